// Tensor-core split-KV attention under the hybrid mask for sm_100a: TMA-staged KV pages,
// tcgen05 MMAs with accumulators in tensor memory, softmax in registers.
//
// Work decomposition.  The plan kernel cuts every sequence's query block into row blocks (as many
// block rows as fit a 128-row tile with their G q-heads; one per sequence unless the block is long),
// numbers all 128-token KV tiles of the call (row block, then kv-head, then position) and cuts them
// into one contiguous range per persistent CTA, of equal cost (tiles plus a start-up charge per
// segment).  A range is walked piece by piece, a piece being its intersection with one
// (row block, kv-head) segment.
//
// One piece.  The at most 128 query rows of a row block that share the kv-head (row r = block row
// r / G of q-head kvh * G + r % G) form the M = 128 operand of every MMA, so each KV tile is
// read from HBM once for all of them.  Per tile j of the piece:
//     producer warps: one for K, one for V; 8 lanes issue one TMA box each -- a whole page of the
//                     kv-head, both 64-wide halves of d (4 KB: the TMA unit's cost is mostly per
//                     box, measured 20.9 B/clk per SM with 2 KB boxes, 28.9 with 4 KB) -- into a
//                     128B-swizzled buffer [8-token group][half][8 rows][128 B] of a 3-deep ring
//                     per operand; a K buffer is released by the QK^T commit, a V buffer by P V;
//     MMA warp      : S_s = Q K^T (tcgen05.mma, A and B from shared memory, S in TMEM), and
//                     after the softmax O_s += P_s V (A = P from TMEM, B = V MN-major);
//     softmax group : 128 threads, one query row each: tcgen05.ld the row of S, hybrid mask
//                     from the row's (kind, index) -> first invisible key position, online
//                     softmax in the log2 domain, bf16 P written back over S in TMEM.
// Tiles alternate between two independent streams s = j & 1, each with its own softmax
// group, S/P buffer, (m, l) state and O accumulator in TMEM, so the tensor pipe works on one
// stream while the other is in its softmax; the two streams are merged in the epilogue.  A segment
// that several CTAs share is merged by whichever of them delivers its partial last (a counter, no waiting).  O is
// rescaled lazily (only when a row maximum grows by more than 2^8), which is exact because
// the same reference maximum is used for P, l and O.
//
// TMEM columns: S0/P0 [0,128)  S1/P1 [128,256)  O0 [256,256+d)  O1 [384,384+d).
//
// Pieces are pipelined as well: every role walks the CTA's pieces on its own and meets the others only
// through mbarriers.  The load warps run ahead through the K / V rings; a fourth helper warp brings
// the next piece's Q tile in (TMA) as soon as the last QK^T of the current piece has completed, has
// the piece after that prefetched into L2, and publishes every piece's descriptor for the MMA warp and
// the softmax groups; the MMA warp starts the next piece while the softmax groups are still in the
// epilogue of the current one (the first P V of a piece waits until the epilogue has read O).
//
// Every wait is bounded.  A wait that runs out raises a CTA-wide abort flag: all roles leave
// their loops, in-flight TMA copies are drained, TMEM is released and FD_DEV_TIMEOUT is set.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <vector>

#include "fd_internal.cuh"
#include "fd_sm100.cuh"

namespace fd {

using namespace sm100;

namespace {

constexpr int kThreads = 384;  // warps 0-3 softmax group 0, 4-7 softmax group 1, 8 K loads, 9 V loads, 10 MMA, 11 Q loads
constexpr int kKWarp = 8, kVWarp = 9, kMmaWarp = 10;  // warp 11 loads Q
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kEarlyLoadMaxTiles = 96;     // longest range of a CTA that starts on its KV before the previous launch has completed
// Who issues the P V of a tile.  In a range of at least kGroupPvMinTiles tiles warp 0 of the softmax group that wrote P
// issues it, as soon as the group's P is whole: the MMA warp, which takes its waits in program order (K tile, then the
// P V that last read the S buffer), then never stands between a finished P and its P V (3-10 % per call from batch 8
// upwards).  In a shorter range -- and in the cluster form, whose CTAs have one to three tiles -- the MMA warp issues
// it: there the issue sits on the group's critical path for nothing (batch 1: +0.7 us per call when tried).
#ifndef FD_GROUP_PV_MIN_TILES
#define FD_GROUP_PV_MIN_TILES 6
#endif
constexpr int kGroupPvMinTiles = FD_GROUP_PV_MIN_TILES;
template <int MODE>
__device__ __forceinline__ bool pv_by_group(int range_tiles) { return MODE != kTcCluster && range_tiles >= kGroupPvMinTiles; }

// 1: Q K^T(j) waits for the completion of the P V whose P it overwrites; 0: it does not (see mma_role).
#ifndef FD_QK_MODE
#define FD_QK_MODE 1
#endif
// 1: the first fill of the K and V rings is staggered (see load_role)
#ifndef FD_STAGGER
#define FD_STAGGER 1
#endif

template <int D, int MODE>
struct Cfg {
    static constexpr int kStages = (D == 128) ? 3 : 6;   // buffers in the K ring, and again in the V ring
    static constexpr int kQBytes = kMaxRows * D * 2;
    static constexpr int kKBytes = kTileTokens * D * 2;  // one K (or V) tile
    static constexpr int kBarOffset = kQBytes + 2 * kStages * kKBytes;
    static constexpr int kCsOffset = kBarOffset + 320;           // window of the CTA range starts
    static constexpr int kDescOffset = kBarOffset + 448;         // ring of piece descriptors
    static constexpr int kScanOffset = kBarOffset + 720;         // SelfScans: the scans of a call that plans for itself
    static constexpr int kExOffset = kBarOffset + 1024;          // [2][128] floats: stream exchange in the epilogue
    static constexpr int kRbOffset = kBarOffset + 2048;          // row blocks of a call that plans for itself
    static constexpr int kSmemBytes = kBarOffset + 3072;         // the dynamic shared memory is declared 1024-byte aligned
    static constexpr int kKSteps = D / 16;
    static constexpr int kHalves = D / 64;
    // A K or V tile in shared memory: [8-token group][half of d][8 rows][128 B] -- what one TMA box per page
    // (two groups) lands; for either half the 16 groups lie kGroupBytes apart, the stride the MMA descriptors name.
    static constexpr int kGroupBytes = kHalves * 1024;
    static constexpr int kPageBytes = 2 * kGroupBytes;
};

struct Bars {
    uint64_t k_full[6], k_empty[6], v_full[6], v_empty[6];
    uint64_t s_full[2], p_full[2], pv_done[2];
    uint64_t q_full, q_free;   // Q tile of a piece landed / no longer read by any MMA
    uint64_t o_free;           // the epilogue of a piece has read O out of TMEM
    uint64_t merge_bar;        // the other pieces of a segment have been copied into shared memory (merger, last piece)
    uint32_t tmem_base;
    int abort;
    int epi_flag;              // per-epilogue decisions of thread 0: bit 0 merge, bit 1 leave
    int desc_n;                // piece descriptors published so far (written by the Q load warp)
    int piece_ok;              // thread 0 of the softmax groups: the descriptor of the next piece is there
    int first;                 // a call that plans for itself: the row block that owns the first tile of this CTA's range
    int bad;                   // a load warp of this CTA met a page id outside the pool
};
constexpr int kDescSlots = 4;

// The plan of a call that plans for itself (at most kSelfPlanMaxRb sequences, one row block each), in shared memory.
struct SelfScans {
    int cu_q[kSelfPlanMaxRb + 1], cu_tiles[kSelfPlanMaxRb + 1], cu_ne[kSelfPlanMaxRb + 1];
    int fatal;
};
static_assert(sizeof(SelfScans) <= 304, "SelfScans must fit between the descriptor ring and the exchange buffer");
static_assert(sizeof(RowBlock) * kSelfPlanMaxRb <= 1024, "row blocks of a self-planned call must fit their slot");

// The tiles [s_c, e_c) a CTA works on and the row block that owns the first of them.
struct Range {
    int s_c, e_c, first;
};
static_assert(sizeof(Bars) <= 320, "Bars must fit in front of the range-start window");

struct Piece {
    int v, b, kvh, tile0, nt, n, Lq, M, nb, i0, Lv, kv_len, rows, row0, slot, seg_nt;  // v: row block; Lv: its block rows
    bool complete;
};

// Piece that starts at tile t.  `hint` is a row block at or before the one that owns t (pieces are walked in
// order, so the previous piece's row block will do): a short forward walk replaces a search.
__device__ __forceinline__ Piece decode_piece(const AttnParams& p, int n_rb, int t, int s_c, int e_c, int cta, int hint) {
    // p.plan may point into shared memory (a call that plans for itself): plain loads either way
    Piece pc;
    int lo = hint;
    while (lo + 1 < n_rb && p.Hkv * p.plan.cu_tiles[lo + 1] <= t) ++lo;
    pc.v = lo;
    const int ntiles = p.plan.cu_tiles[lo + 1] - p.plan.cu_tiles[lo];
    const int rem = t - p.Hkv * p.plan.cu_tiles[lo];
    pc.kvh = rem / ntiles;
    pc.tile0 = rem % ntiles;
    const int seg_start = t - pc.tile0, seg_end = seg_start + ntiles;
    const int t_end = min(e_c, seg_end);
    pc.nt = t_end - t;
    pc.seg_nt = ntiles;
    const int4* rbp = reinterpret_cast<const int4*>(p.plan.rb + lo);
    const int4 r0 = rbp[0], r1 = rbp[1];  // (b, i0, n, Lq), (M, nb, -, -)
    pc.b = r0.x;
    pc.i0 = r0.y;
    pc.n = r0.z;
    pc.Lq = r0.w;
    pc.M = r1.x;
    pc.nb = r1.y;
    pc.Lv = min(p.rb_rows, pc.Lq - pc.i0);
    pc.kv_len = pc.n + pc.Lq;
    pc.rows = pc.Lv * p.G;
    pc.row0 = p.plan.cu_q[lo];
    // with one cluster per segment every piece goes through the cluster merge, a piece that holds all tiles too
    pc.complete = (t == seg_start) && (t_end == seg_end) && p.cluster == 0;
    pc.slot = 2 * cta + (t == s_c ? 0 : 1);
    return pc;
}


__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Under programmatic dependent launch: block until the launch before this one on the stream has completed and its
// writes are visible.  Returns at once when that has happened already (or the launch was an ordinary one).
__device__ __forceinline__ void wait_prior_launch() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Warp-uniform bounded wait.
__device__ __forceinline__ bool wait_all(uint64_t* bar, uint32_t parity, volatile int* abort) {
    const bool ok = mbar_wait(bar, parity, abort);
    return __all_sync(0xffffffffu, ok);
}

// Piece descriptors.  The Q load warp walks the pieces ahead of everyone, decodes each one (a chain of
// dependent global loads) and publishes it in a small ring in shared memory; the MMA warp and the softmax
// groups pick it up from there, so the decode is off their critical path at a piece boundary.  Slot
// reuse is safe: descriptor N + 1 is written after every QK^T of piece N - 1 has completed, when no
// consumer is before piece N - 1 and every consumer copies its descriptor to registers at piece start.
__device__ __forceinline__ void publish_piece(Bars* bars, Piece* ring, int n, const Piece& pc) {
    ring[n & (kDescSlots - 1)] = pc;
    asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(&bars->desc_n)), "r"(n + 1) : "memory");
}
__device__ __forceinline__ bool piece_published(Bars* bars, int n) {
    int v;
    asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(&bars->desc_n)) : "memory");
    return v > n;
}
// Bounded like every other wait; false if it gave up (abort raised here or elsewhere).
__device__ __forceinline__ bool wait_piece(Bars* bars, int n, volatile int* abort) {
    if (piece_published(bars, n)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (piece_published(bars, n)) return true;
        if ((it & 15u) == 0u) {
            if (*abort) return false;
            if (global_ns() - t0 > kWaitLimitNs) break;
        }
    }
    *abort = 1;
    return false;
}

// ---------------------------------------------------------------------------------------------
// Roles.  Each walks the pieces of the CTA's tile range [s_c, e_c) in the same order and keeps
// its own copies of the running counters:
//   g0        KV tiles pushed through the rings before this piece      (ring slot and phase)
//   u_base[s] tiles stream s has processed before this piece           (phase of s_full / p_full / pv_done)
//   piece     pieces before this one                                   (phase of q_full / q_free / o_free)
// ---------------------------------------------------------------------------------------------
struct Walk {
    int t, g0, u_base[2], piece, b;
    __device__ __forceinline__ void advance(const Piece& pc) {
        b = pc.v;  // the row block: the next piece's walk starts from it
        g0 += pc.nt;
        u_base[0] += (pc.nt + 1) >> 1;
        u_base[1] += pc.nt >> 1;
        ++piece;
        t += pc.nt;
    }
};

// K (which = 0) or V (which = 1) load warp.
template <int D, int MODE>
__device__ __forceinline__ void load_role(const CUtensorMap& tmap, const AttnParams& p, int n_rb, unsigned char* ring, uint64_t* full,
                                          uint64_t* empty, int which, const Range rg, uint64_t* k0_full, volatile int* bad, volatile int* abort) {
    using C = Cfg<D, MODE>;
    const int lane = threadIdx.x & 31, cta = blockIdx.x;
    constexpr int kOps = 8;  // pages of a tile: one box each
    const int pg = lane;
    int issued = 0;
    // the KV stream is read once: let it leave L2 first, so that Q, the split partials and the page
    // table (all re-read) stay resident next to a stream many times the size of the cache
    const uint64_t policy = make_policy_evict_first();
    const int s_c = rg.s_c, e_c = rg.e_c;
    Walk w = {s_c, 0, {0, 0}, 0, rg.first};
    bool ok = true;
    // p.early: the first piece and its first page ids are looked up while the launch before this one may still run;
    // p.early == 2: so is the KV pool itself -- that launch is known not to write it -- and this warp waits for it
    // only if it has something to write (a sequence to flag); p.early == 3: that launch is the KV append, which
    // writes the query block's own slots and nothing else: tiles of the prefix are read ahead, the wait comes before
    // the first tile that reaches into the block (pages are 16 tokens, tiles 128: no page lies in both kinds)
    bool waited = !p.early;
    int bad_early = -1;
    while (w.t < e_c && ok) {
        const Piece pc = decode_piece(p, n_rb, w.t, s_c, e_c, cta, w.b);
        const int32_t* table = p.page_table + (long long)pc.b * p.max_pages;
        // Page ids are fetched a batch of four tiles (32 pages, one per lane) at a time and one batch
        // ahead, so the table lookup -- a dependent global load -- never sits between a buffer becoming
        // free and its refill, not even while the ring is filling up at the start of a piece.
        auto load_ids = [&](int batch) -> int {
            const int j = batch * 4 + (lane >> 3);
            const int pos = ((pc.tile0 + j) * 8 + (lane & 7)) * 16;
            if (!(j < pc.nt && pos < pc.kv_len)) return -1;
            int id = table[pos >> 4];
            if ((unsigned)id >= (unsigned)p.num_pages) {  // never form an address from a bad id
                if (!waited && p.early >= 2) { wait_prior_launch(); waited = true; }
                if (waited) flag_sequence(p, pc.b); else bad_early = pc.b;  // (no global write ahead of the prior launch)
                *bad = 1;
                id = 0;
            }
            return id;
        };
        int ids_cur = load_ids(0), ids_next = load_ids(1);
        for (int j = 0; j < pc.nt; ++j) {
            const int g = w.g0 + j, st = g % C::kStages, use = g / C::kStages;
            if (j > 0 && (j & 3) == 0) { ids_cur = ids_next; ids_next = load_ids((j >> 2) + 1); }
            const int phys = __shfl_sync(0xffffffffu, ids_cur, (j & 3) * 8 + pg);
            if (!waited && (p.early == 1 || (p.early == 3 && (pc.tile0 + j + 1) * kTileTokens > pc.n))) {  // the launch before this one may write what this tile holds
                wait_prior_launch();
                waited = true;
                if (bad_early >= 0) flag_sequence(p, bad_early);
            }
            if (!wait_all(&empty[st], (use & 1) ^ 1, abort)) { ok = false; break; }
#if FD_STAGGER
            // The first fill of the rings is not issued all at once: every CTA of the grid starts at the same moment,
            // and 224 KB per SM in one burst makes the first K tile -- all the MMA warp needs to begin -- land with
            // the last of it.  K tiles 0 and 1 go out at once; the V tiles and the third K tile follow when K tile 0
            // has landed (V tile 0 is not needed before the first softmax is through).  A delay, not a dependency:
            // it ends by itself after a few microseconds.
            if (g == (which ? 0 : 2) && k0_full != nullptr) {
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(k0_full, 0) && global_ns() - t0 < 4000ull) {}
                __syncwarp();
            }
#endif
            const int pos0 = (pc.tile0 + j) * kTileTokens;
            const int npg = min(8, (pc.kv_len - pos0 + 15) >> 4);
            if (lane == 0) mbar_arrive_expect_tx(&full[st], npg * (16 * D * 2));
            __syncwarp();
            if (lane < kOps && phys >= 0) {
                unsigned char* dst = ring + st * C::kKBytes + pg * C::kPageBytes;
                tma_load_4d_hint(dst, &tmap, 0, 0, 0, ((phys * 2 + which) * p.Hkv + pc.kvh) * 2, &full[st], policy);
            }
            issued = g + 1;
        }
        w.advance(pc);
    }
    if (*abort) {  // drain TMA copies still in flight before the shared memory is given back
        for (int g = max(0, issued - C::kStages); g < issued; ++g) {
            const int st = g % C::kStages, use = g / C::kStages;
            const unsigned long long t0 = global_ns();
            for (uint32_t it = 0; it < kSpinLimit && global_ns() - t0 < kWaitLimitNs; ++it)
                if (mbar_try_wait(&full[st], use & 1)) break;
        }
    }
}

// Q load warp: the G * Lq rows of a piece -> shared memory, K-major, 128-byte swizzle.  q is seen as
// [T][Hq][d]; one TMA box is 64 elements of d x the G q-heads of the kv-head x q_box_t block rows, which
// lands as q_box_t * G consecutive 128-byte rows, row (i, g) at i * G + g: the order the MMA wants.  The
// last box of a piece may reach past the block (rows of the next sequence, or zeros past T): each query
// row only ever influences its own output row, and those rows are never stored.
template <int D, int MODE>
__device__ __forceinline__ void q_role(const CUtensorMap& qmap, const AttnParams& p, int n_rb, unsigned char* sq, Bars* bars, Piece* ring,
                                       const Range rg, volatile int* abort) {
    using C = Cfg<D, MODE>;
    const int lane = threadIdx.x & 31, cta = blockIdx.x;
    const int bt = p.q_box_t;
    const int s_c = rg.s_c, e_c = rg.e_c;
    Walk w = {s_c, 0, {0, 0}, 0, rg.first};
    int issued = 0;
    Piece pc = decode_piece(p, n_rb, w.t, s_c, e_c, cta, w.b);
    if (lane == 0) publish_piece(bars, ring, 0, pc);
    if (p.early == 1) wait_prior_launch();  // q may be written by it (p.early >= 2: it is known not to be)
    while (w.t < e_c) {
        if (w.piece > 0 && !wait_all(&bars->q_free, (w.piece - 1) & 1, abort)) break;
        const int nbox = (pc.Lv + bt - 1) / bt;
        if (lane == 0) mbar_arrive_expect_tx(&bars->q_full, nbox * bt * p.G * 128 * C::kHalves);
        __syncwarp();
        for (int e = lane; e < nbox * C::kHalves; e += 32) {
            const int j = e / C::kHalves, half = e % C::kHalves;
            tma_load_3d(sq + half * (kMaxRows * 128) + j * bt * p.G * 128, &qmap, half * 64, pc.kvh * p.G, pc.row0 + j * bt, &bars->q_full);
        }
        issued = w.piece + 1;
        w.advance(pc);
        if (w.t < e_c) {
            // the next piece: descriptor for the other roles, and its Q rows on their way into L2
            pc = decode_piece(p, n_rb, w.t, s_c, e_c, cta, w.b);
            if (lane == 0) publish_piece(bars, ring, w.piece, pc);
            const int nb2 = (pc.Lv + bt - 1) / bt;
            for (int e = lane; e < nb2 * C::kHalves; e += 32)
                tma_prefetch_3d(&qmap, (e % C::kHalves) * 64, pc.kvh * p.G, pc.row0 + (e / C::kHalves) * bt);
        }
    }
    if (*abort && issued > 0) {  // drain the last copy before the shared memory is given back
        const unsigned long long t0 = global_ns();
        for (uint32_t it = 0; it < kSpinLimit && global_ns() - t0 < kWaitLimitNs; ++it)
            if (mbar_try_wait(&bars->q_full, (issued - 1) & 1)) break;
    }
}

// A segment's ragged last tile: V rows no token owns may hold NaN or stale data -- P is 0 there, but 0 * NaN is not.
// The warp that is about to issue the tile's P V zeroes them (the tile has landed) and fences the writes for the MMA.
template <class C>
__device__ __forceinline__ void zero_v_tail(unsigned char* vt, int valid, int lane) {
    if (valid >= kTileTokens) return;
    const int nbad = kTileTokens - valid;
    for (int e = lane; e < nbad * 8 * C::kHalves; e += 32) {
        const int r = valid + e / (8 * C::kHalves), wd = e % (8 * C::kHalves);
        *reinterpret_cast<uint4*>(vt + (r >> 3) * C::kGroupBytes + (wd >> 3) * 1024 + (r & 7) * 128 + ((wd & 7) << 4)) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
    __syncwarp();
}

// MMA issuing warp.
template <int D, int MODE>
__device__ __forceinline__ void mma_role(const AttnParams& p, unsigned char* sq, unsigned char* sk, unsigned char* sv, Bars* bars,
                                         const Piece* ring, uint32_t tmem, const Range rg, volatile int* abort) {
    using C = Cfg<D, MODE>;
    const int lane = threadIdx.x & 31;
    constexpr uint32_t idesc_qk = make_idesc_bf16(128, kTileTokens, false);
    constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, true);
    const uint32_t col_s[2] = {0u, 128u}, col_o[2] = {256u, 384u};
    const bool group_pv = pv_by_group<MODE>(rg.e_c - rg.s_c);
    if (p.early == 1) wait_prior_launch();  // (this role touches shared and tensor memory only; p.early >= 2 lets it run ahead)
    const uint64_t qd0 = make_smem_desc(smem_u32(sq), 16, 1024);
    const int s_c = rg.s_c, e_c = rg.e_c;
    Walk w = {s_c, 0, {0, 0}, 0, rg.first};
    bool ok = true;
    while (w.t < e_c && ok) {
        if (!__all_sync(0xffffffffu, wait_piece(bars, w.piece, abort))) break;
        const Piece pc = ring[w.piece & (kDescSlots - 1)];
        if (!wait_all(&bars->q_full, w.piece & 1, abort)) break;
        auto issue_pv = [&](int jj) {  // (ranges whose P V this warp issues: see kGroupPvMinTiles)
            const int gg = w.g0 + jj, s = jj & 1, st = gg % C::kStages, u = w.u_base[s] + (jj >> 1);
            if (!wait_all(&bars->v_full[st], (gg / C::kStages) & 1, abort)) { ok = false; return; }
            unsigned char* vt = sv + st * C::kKBytes;
            zero_v_tail<C>(vt, pc.kv_len - (pc.tile0 + jj) * kTileTokens, lane);
            // the first P V of a stream in a piece overwrites O: the previous piece's epilogue must have read it
            if (jj < 2 && w.piece > 0 && !wait_all(&bars->o_free, (w.piece - 1) & 1, abort)) { ok = false; return; }
            // (descriptors are made before the last wait: what follows it is the MMA instructions alone.  The address
            // field of a descriptor is its low 14 bits, in 16-byte units, so a K step is an addition.)
            const uint64_t vd0 = make_smem_desc(smem_u32(vt), 1024, C::kGroupBytes);
            if (!wait_all(&bars->p_full[s], u & 1, abort)) { ok = false; return; }
            tc_fence_after();
            if (lane == 0) {
#pragma unroll
                for (int kk = 0; kk < kTileTokens / 16; ++kk)
                    // one page per K step: its two 8-token groups lie kGroupBytes apart, the two halves of d 1 KB apart
                    umma_ts(tmem + col_o[s], tmem + col_s[s] + kk * 8, vd0 + (uint64_t)((kk * C::kPageBytes) >> 4), idesc_pv, jj >= 2 || kk > 0);
                umma_commit(&bars->v_empty[st]);
                umma_commit(&bars->pv_done[s]);
            }
            __syncwarp();
        };
        for (int j = 0; j < pc.nt && ok; ++j) {
            const int g = w.g0 + j, st = g % C::kStages, use = g / C::kStages;
            const int s = j & 1;
            if (!wait_all(&bars->k_full[st], use & 1, abort)) { ok = false; break; }
            // S_s is written over P_s (its first 64 columns), which the P V of tile j - 2 of this stream reads, and
            // nothing orders two MMAs with different accumulators but the completion of the first: Q K^T waits for
            // that P V's completion barrier.  (FD_QK_MODE 0 drops the wait, relying on one thread's MMAs executing in
            // issue order: 3-5 % faster, but not a documented guarantee; kept for measurements only.  Tried as well:
            // Q K^T as two N = 64 halves with only the aliasing half behind the wait, 11 % slower; issuing whichever
            // MMA is ready first from a polling loop, 8 % slower -- the polling warp takes issue slots from the
            // softmax warps of its scheduler.)
            [[maybe_unused]] const int u_prev = w.u_base[s] + (j >> 1) - 1;  // the stream's previous tile, over all pieces
            const uint64_t kd0 = make_smem_desc(smem_u32(sk + st * C::kKBytes), 16, C::kGroupBytes);
#if FD_QK_MODE != 0
            if (u_prev >= 0 && !wait_all(&bars->pv_done[s], u_prev & 1, abort)) { ok = false; break; }
#endif
            tc_fence_after();
            if (lane == 0) {
#pragma unroll
                for (int kk = 0; kk < C::kKSteps; ++kk) {
                    constexpr int kQHalf = kMaxRows * 128;
                    umma_ss(tmem + col_s[s], qd0 + (uint64_t)(((kk >> 2) * kQHalf + (kk & 3) * 32) >> 4),
                            kd0 + (uint64_t)(((kk >> 2) * 1024 + (kk & 3) * 32) >> 4), idesc_qk, kk > 0);
                }
                umma_commit(&bars->k_empty[st]);
                umma_commit(&bars->s_full[s]);
                if (j == pc.nt - 1) umma_commit(&bars->q_free);  // the next piece's Q may come in
            }
            __syncwarp();
            if (!group_pv && j >= 1) issue_pv(j - 1);
        }
        if (!group_pv && ok) issue_pv(pc.nt - 1);
        w.advance(pc);
    }
}

// ---------------------------------------------------------------------------------------------
// One cluster per segment (kTcCluster).  The CTAs of a cluster split the segment's tiles evenly.  Query row r of the
// segment is owned by CTA r / share of the cluster (share = ceil(128 / cluster size)).  Every CTA writes the
// unnormalised partial result of the rows it does not own -- O in fp32 and (m, l) -- to its two scratch slots in
// global memory, one block per owner, keeps the rows it owns in registers, and after ONE cluster barrier each owner
// brings the c - 1 blocks meant for it into its shared memory with bulk copies, combines them with its own part in
// rank order (fixed, so the result does not depend on timing) and writes the bf16 rows.  The cluster is there for the
// barrier and the co-scheduling; the bytes go through L2, because that is the faster carrier: an SM stores 64 KB to
// global memory in 0.9 us and a bulk copy lands it in 0.3 us, while the SM-to-SM path moved the same rows at about
// 20 GB/s per SM (3.5-5 us), with st.shared::cluster pushes as with ld.shared::cluster pulls.  No counters, no polling.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {  // every thread of every CTA of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
constexpr int kMaxCluster = 16;
// Rows a CTA of a cluster of c owns (the last CTA may own fewer, or none).
__host__ __device__ constexpr int cluster_share(int c) { return (kMaxRows + c - 1) / c; }
// What one CTA hands one owner: the O rows as [d / 4 words][share rows][16 bytes], then (m, l) per row.
__host__ __device__ constexpr uint32_t cluster_block_bytes(int c, int d) { return (uint32_t)((cluster_share(c) * (d * 4 + 8) + 15) / 16 * 16); }
// Do the two scratch slots of a CTA, and the K ring where the blocks land, hold the c blocks of a cluster of c?
__host__ __device__ constexpr bool cluster_fits(int c, int d) {
    return (uint32_t)c * cluster_block_bytes(c, d) <= 2u * kMaxRows * d * 4 &&
           (uint32_t)c * cluster_block_bytes(c, d) <= (uint32_t)(d == 128 ? 3 : 6) * kTileTokens * d * 2;
}

// Addresses of the exchange.  In global memory: CTA `cta` of the grid owns scratch slots 2 cta and 2 cta + 1, one block
// per owner rank.  In shared memory: after the cluster barrier the K ring (idle by then) takes the c blocks meant for
// this CTA, block c from rank c; its own block it has written there itself.
template <int D>
struct Exchange {
    unsigned char* g_base;  // scratch of this CTA
    unsigned char* land;    // the K ring (generic address)
    uint32_t land_s;        // ... and its shared-memory address
    int share;
    uint32_t block;
    __device__ __forceinline__ unsigned char* g_block(int dest) const { return g_base + (size_t)dest * block; }
    __device__ __forceinline__ static uint32_t o_off(int share_, int rl, int word) { return (uint32_t)(word * share_ + rl) * 16; }
    __device__ __forceinline__ uint32_t ml_off(int rl) const { return (uint32_t)share * D * 4 + (uint32_t)rl * 8; }
};

// Owner side, after the cluster barrier: warp 0 brings the peers' blocks in, a lane per peer.
template <int D>
__device__ __forceinline__ void cluster_fetch(const AttnParams& p, const Exchange<D>& ex, Bars* bars, int rank) {
    const int C = p.cluster, c = threadIdx.x & 31;
    if (c == 0) mbar_arrive_expect_tx(&bars->merge_bar, (uint32_t)(C - 1) * ex.block);
    __syncwarp();
    if (c < C && c != rank) {
        fence_proxy_async_all();  // the peers' plain stores, acquired at the barrier, before the bulk copy that reads them
        const long long cta_stride = (long long)2 * kMaxRows * D * 4;  // two scratch slots per CTA
        bulk_load(ex.land + (size_t)c * ex.block, ex.g_base + (c - rank) * cta_stride + (long long)rank * ex.block, ex.block, &bars->merge_bar);
    }
}

// Owner side, once the blocks have landed: the eight warps of the softmax groups share the rows this CTA owns, a row
// per D / 4 lanes, a lane per 16-byte word (its 8-byte bf16 stores form one contiguous run per row).  Lane c of a row's
// group holds part c's (m, l) and weight, handed round by shuffles; the c parts are combined in rank order.
template <int D>
__device__ __forceinline__ void cluster_reduce(const AttnParams& p, const Exchange<D>& ex, int rank, int rows, int kvh, int row0) {
    constexpr int kLpr = D / 4;              // lanes per row (>= the largest cluster)
    constexpr int kRowsPerWarp = 32 / kLpr;
    static_assert(kLpr >= kMaxCluster, "one lane per part");
    const int C = p.cluster, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int word = lane % kLpr;
    const int r_lo = rank * ex.share, n_own = min(ex.share, rows - r_lo);  // rows [r_lo, r_lo + n_own) are this CTA's
    for (int rl0 = 0; rl0 < n_own; rl0 += 8 * kRowsPerWarp) {              // uniform over the warp: it shuffles
        const int rl = rl0 + warp * kRowsPerWarp + lane / kLpr;
        const bool act = rl < n_own;
        const int rl_c = act ? rl : 0;
        float2 q = make_float2(-INFINITY, 0.f);
        if (act && word < C) q = *reinterpret_cast<const float2*>(ex.land + (size_t)word * ex.block + ex.ml_off(rl_c));
        float m = q.x;
        int flagged = q.y < 0.f;  // some CTA of the cluster met a page id outside the pool (it sent l < 0)
#pragma unroll
        for (int o = kLpr / 2; o > 0; o >>= 1) {
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o, kLpr));
            flagged |= __shfl_xor_sync(0xffffffffu, flagged, o, kLpr);
        }
        const float w = q.x == -INFINITY ? 0.f : exp2f(q.x - m);  // a part that saw no visible key for the row counts nothing
        float l = w * q.y;
#pragma unroll
        for (int o = kLpr / 2; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o, kLpr);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        const unsigned char* o0 = ex.land + Exchange<D>::o_off(ex.share, rl_c, word);
        for (int c0 = 0; c0 < C; c0 += 4) {
            float4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] = *reinterpret_cast<const float4*>(o0 + (size_t)min(c0 + k, C - 1) * ex.block);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float wc = __shfl_sync(0xffffffffu, w, min(c0 + k, C - 1), kLpr);
                if (c0 + k < C && wc != 0.f) {  // (by selection: the O rows of a part without weight may hold anything)
                    acc.x += wc * v[k].x; acc.y += wc * v[k].y; acc.z += wc * v[k].z; acc.w += wc * v[k].w;
                }
            }
        }
        if (!act) continue;
        float inv = l > 0.f ? 1.f / l : 0.f;
        if (flagged) {  // by assignment: what came from a stand-in page may be inf or NaN
            inv = 0.f;
            acc = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const int r = r_lo + rl;
        __nv_bfloat16* dst = p.out + ((long long)(row0 + r / p.G) * p.Hq + kvh * p.G + r % p.G) * D + word * 4;
        __align__(8) __nv_bfloat162 v2[2] = {__floats2bfloat162_rn(acc.x * inv, acc.y * inv), __floats2bfloat162_rn(acc.z * inv, acc.w * inv)};
        *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(v2);
    }
}

// Merge of a split segment from shared memory (the merger at the last piece of its range, when the Q tile and the
// rings are idle).  The staging area holds kRound O arrays of partial slots ([D / 4][128 rows][4 floats]) and behind
// them the (m[128], l[128]) pairs: first this CTA's own, then those of the n_other other pieces in CTA order.  The O
// arrays come in rounds of kRound pieces (bulk copies issued by thread 0 through issue_round, completion on merge_bar);
// this CTA's own piece -- the own_pos-th of the segment in CTA order -- is in registers (own: the thread's D / 2
// columns).  Same arithmetic, same order as merge_row: the result does not depend on who merges.  Called by all 256
// threads of the softmax groups (it holds barriers); `active`: the thread has a row to write.
template <int D, int MODE>
struct Stage {
    static constexpr uint32_t kBytes = Cfg<D, MODE>::kQBytes + 2 * Cfg<D, MODE>::kStages * Cfg<D, MODE>::kKBytes;
    static constexpr uint32_t kPieceBytes = kMaxRows * D * 4;
    static constexpr int kRound = (kBytes - 8192) / kPieceBytes;
    static constexpr uint32_t kMlOffset = kRound * kPieceBytes;
    static constexpr int kMaxOthers = (kBytes - kMlOffset) / (2 * kMaxRows * 4) - 1;
};

template <int D, int MODE, class IssueRound>
__device__ __forceinline__ void merge_staged(const AttnParams& p, Bars* bars, const unsigned char* stage, int n_other, int own_pos,
                                             const float* own, int r, int cg, bool active, bool flagged, int kvh, int row0,
                                             volatile int* abort, IssueRound issue_round) {
    using S = Stage<D, MODE>;
    constexpr int CW = D / 2;
    const float* ml = reinterpret_cast<const float*>(stage + S::kMlOffset);  // [1 + n_other][2][128]
    float acc[CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) acc[c] = 0.f;
    float m = -INFINITY, l = 0.f;
    auto add_own = [&]() {
        const float mp = ml[r], lp = ml[kMaxRows + r];
        const float w = (mp == -INFINITY) ? 0.f : exp2f(mp - m);
        l += w * lp;
#pragma unroll
        for (int k = 0; k < CW; ++k) acc[k] += w * own[k];
    };
    for (int round = 0, k0 = 0;; ++round, k0 += S::kRound) {
        if (!wait_all(&bars->merge_bar, round & 1, abort)) return;  // uniform: every thread sees the same outcome or leaves
        if (round == 0 && active) {
            m = ml[r];
            for (int k = 0; k < n_other; ++k) m = fmaxf(m, ml[(1 + k) * 2 * kMaxRows + r]);
        }
        const int k1 = min(n_other, k0 + S::kRound);
        if (active) {
            for (int k = k0; k < k1; ++k) {
                if (k == own_pos) add_own();
                const float mp = ml[(1 + k) * 2 * kMaxRows + r], lp = ml[(1 + k) * 2 * kMaxRows + kMaxRows + r];
                const float w = (mp == -INFINITY) ? 0.f : exp2f(mp - m);
                l += w * lp;
                const float4* o = reinterpret_cast<const float4*>(stage + (size_t)(k - k0) * S::kPieceBytes) + ((cg * CW) >> 2) * kMaxRows + r;
#pragma unroll
                for (int q = 0; q < CW / 4; ++q) {
                    const float4 v = o[q * kMaxRows];
                    acc[4 * q] += w * v.x;
                    acc[4 * q + 1] += w * v.y;
                    acc[4 * q + 2] += w * v.z;
                    acc[4 * q + 3] += w * v.w;
                }
            }
        }
        if (k1 == n_other) break;
        named_bar_sync(1, 256);  // everyone has read this round's O arrays: the next round may land on them
        if (threadIdx.x == 0) issue_round(round + 1);
    }
    if (!active) return;
    if (own_pos == n_other) add_own();
    __nv_bfloat16* dst = p.out + ((long long)(row0 + r / p.G) * p.Hq + kvh * p.G + r % p.G) * D + cg * CW;
    if (flagged) {  // a page id of this sequence was bad: defined output, zeros (by assignment)
#pragma unroll
        for (int c = 0; c < CW; ++c) acc[c] = 0.f;
        store_cols_bf16<CW>(dst, acc, 0.f);
        return;
    }
    store_cols_bf16<CW>(dst, acc, 1.f / l);
}

// The two softmax groups (256 threads).
template <int D, int MODE>
__device__ __forceinline__ void softmax_role(const AttnParams& p, Bars* bars, float* ex, int* s_cs, const CtaStarts cs, const Piece* ring,
                                             uint32_t tmem, const Range rg, const Exchange<D> exch, int cl_rank, unsigned char* stage,
                                             unsigned char* sv, volatile int* abort) {
    using C = Cfg<D, MODE>;
    constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, true);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, cta = blockIdx.x;
    const int s_c = rg.s_c, e_c = rg.e_c;
    const int s = warp >> 2;                  // stream
    const int r = (warp & 3) * 32 + lane;     // query row == TMEM lane
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t col_s[2] = {0u, 128u}, col_o[2] = {256u, 384u};
    const float c = p.scale_log2e;
    // fill the window of range starts; the barrier below orders it before its first use
    if (MODE == kTcPlanned && tid < kCsWindow) {  // (a call that plans for itself has filled it while planning)
        const int cc = cs.base + tid;
        s_cs[tid] = (cc >= 0 && cc <= p.n_ctas) ? cs.g[cc] : 0;
    }
    bool cl_synced = false;
    // before any global write of this role (scratch, counters, out).  p.early == 2: the tiles of the first piece may be
    // worked through meanwhile -- tensor and shared memory only -- and the wait comes before its ticket and epilogue
    if (p.early == 1) wait_prior_launch();
    bool prior_done = p.early < 2;
    const bool group_pv = pv_by_group<MODE>(e_c - s_c);
    Walk w = {s_c, 0, {0, 0}, 0, 0};
    while (w.t < e_c) {
        // one thread waits for the descriptor, so that all 256 take the same decision
        if (tid == 0) bars->piece_ok = wait_piece(bars, w.piece, abort);
        named_bar_sync(1, 256);
        if (!bars->piece_ok) break;
        const Piece pc = ring[w.piece & (kDescSlots - 1)];
        const bool warp_active = (warp & 3) * 32 < pc.rows;
        const int i = r / p.G;
        const RowMask rm = row_mask(pc.i0 + i, pc.n, pc.Lq, pc.M, pc.nb, r < pc.rows);
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        // Warps whose 32 rows are all padding do nothing per tile: warp 0 of the group (always active)
        // arrives on p_full for them, and they wait at the epilogue's hardware barrier, not by polling.
        const int n_idle_threads = 32 * (4 - min(4, (pc.rows + 31) >> 5));

        for (int j = s; j < pc.nt && warp_active; j += 2) {
            const int u = w.u_base[s] + (j >> 1);
            if (!wait_all(&bars->s_full[s], u & 1, abort)) { ok = false; break; }
            tc_fence_after();
            {
                const int pos0 = (pc.tile0 + j) * kTileTokens;
                // tile reaches into the query block (or past kv_len): the row's mask applies, in tile-local columns
                const bool masked = pos0 + kTileTokens > pc.n;
                const int lim = rm.limit - pos0, blo = rm.blk_lo - pos0, bhi = rm.blk_hi - pos0;
                const uint32_t s_addr = tmem + lane_base + col_s[s];

                // ---- the whole row of S in one round trip: TMEM loads queue behind the MMAs in flight,
                //      so every ld -> wait pair costs up to one MMA tile; registers come from setmaxnreg
                uint32_t sv[4][32];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) tmem_ld32(s_addr + ch * 32, sv[ch]);
                tc_wait_ld();
                if (masked) {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            if (ch * 32 + k >= lim && (ch * 32 + k < blo || ch * 32 + k >= bhi)) sv[ch][k] = 0xff800000u;  // -inf by select: S may be NaN there
                }
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // three-input max: 64 instructions per row
#pragma unroll
                for (int ch = 0; ch < 4; ++ch)
#pragma unroll
                    for (int k = 0; k < 32; k += 8) {
                        mx[0] = max3(mx[0], __uint_as_float(sv[ch][k]), __uint_as_float(sv[ch][k + 1]));
                        mx[1] = max3(mx[1], __uint_as_float(sv[ch][k + 2]), __uint_as_float(sv[ch][k + 3]));
                        mx[2] = max3(mx[2], __uint_as_float(sv[ch][k + 4]), __uint_as_float(sv[ch][k + 5]));
                        mx[3] = max3(mx[3], __uint_as_float(sv[ch][k + 6]), __uint_as_float(sv[ch][k + 7]));
                    }
                const float m_new = fmaxf(m, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c);
                float alpha = 1.f;
                if (j < 2 || m == -INFINITY) {
                    m = m_new;  // nothing accumulated yet (O is overwritten, or exactly zero)
                } else if (m_new > m + kRescaleThreshold) {
                    alpha = exp2f(m - m_new);
                    m = m_new;
                }
                if (__any_sync(0xffffffffu, alpha != 1.f)) {
                    // previous PV of this stream has completed (S/P buffer reuse orders it), so O is quiescent
#pragma unroll 1
                    for (int ch = 0; ch < D / 16; ++ch) {
                        uint32_t o[16];
                        tmem_ld16(tmem + lane_base + col_o[s] + ch * 16, o);
                        tc_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                        tmem_st16(tmem + lane_base + col_o[s] + ch * 16, o);
                    }
                    l *= alpha;
                }

                // ---- P = exp2(S * c - m), row sum, bf16 P written over S (64 tokens -> 32 columns)
                const float mc = (m == -INFINITY) ? 0.f : m;
                const float2 c2 = make_float2(c, c), nm2 = make_float2(-mc, -mc);
                float2 sum0 = make_float2(0.f, 0.f), sum1 = make_float2(0.f, 0.f);
#pragma unroll
                for (int hp = 0; hp < 2; ++hp) {
                    uint32_t pk[32];
#pragma unroll
                    for (int k = 0; k < 32; k += 2) {
                        const float2 xa = __ffma2_rn(make_float2(__uint_as_float(sv[2 * hp][k]), __uint_as_float(sv[2 * hp][k + 1])), c2, nm2);
                        const float2 xb = __ffma2_rn(make_float2(__uint_as_float(sv[2 * hp + 1][k]), __uint_as_float(sv[2 * hp + 1][k + 1])), c2, nm2);
                        const float2 pa = make_float2(ex2_approx(xa.x), ex2_approx(xa.y));
                        const float2 pb = make_float2(ex2_approx(xb.x), ex2_approx(xb.y));
                        sum0 = __fadd2_rn(sum0, pa);
                        sum1 = __fadd2_rn(sum1, pb);
                        const __nv_bfloat162 ba = __floats2bfloat162_rn(pa.x, pa.y), bb = __floats2bfloat162_rn(pb.x, pb.y);
                        pk[k >> 1] = *reinterpret_cast<const uint32_t*>(&ba);
                        pk[16 + (k >> 1)] = *reinterpret_cast<const uint32_t*>(&bb);
                    }
                    tmem_st32(s_addr + hp * 32, pk);  // overwrites S columns that are already in registers
                }
                l += (sum0.x + sum0.y) + (sum1.x + sum1.y);
                tc_wait_st();
            }
            tc_fence_before();
            mbar_arrive(&bars->p_full[s]);
            if ((warp & 3) == 0 && lane == 0 && n_idle_threads) mbar_arrive_cnt(&bars->p_full[s], n_idle_threads);
            if ((warp & 3) == 0 && group_pv) {
                // ---- P V of this tile, issued by warp 0 of the group itself as soon as the group's P is whole: the MMA
                //      warp issues Q K^T only and never stands between a finished P and its P V
                const int gg = w.g0 + j, st = gg % C::kStages;
                unsigned char* vt = sv + st * C::kKBytes;
                if (!wait_all(&bars->v_full[st], (gg / C::kStages) & 1, abort)) { ok = false; break; }
                zero_v_tail<C>(vt, pc.kv_len - (pc.tile0 + j) * kTileTokens, lane);
                // the first P V of a stream in a piece overwrites O: the previous piece's epilogue (both groups) must have read it
                if (j < 2 && w.piece > 0 && !wait_all(&bars->o_free, (w.piece - 1) & 1, abort)) { ok = false; break; }
                // (the address field of a descriptor is its low 14 bits, in 16-byte units, so a K step is an addition)
                const uint64_t vd0 = make_smem_desc(smem_u32(vt), 1024, C::kGroupBytes);
                if (!wait_all(&bars->p_full[s], u & 1, abort)) { ok = false; break; }
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < kTileTokens / 16; ++kk)
                        // one page per K step: its two 8-token groups lie kGroupBytes apart, the two halves of d 1 KB apart
                        umma_ts(tmem + col_o[s], tmem + col_s[s] + kk * 8, vd0 + (uint64_t)((kk * C::kPageBytes) >> 4), idesc_pv, j >= 2 || kk > 0);
                    umma_commit(&bars->v_empty[st]);
                    umma_commit(&bars->pv_done[s]);
                }
                __syncwarp();
            }
        }

        // ---- epilogue: merge the two streams, then final rows, or a partial plus -- if this CTA is the
        //      last one to deliver a piece of the segment -- the merge of all its partials.
        //      All 256 threads take every named barrier, whatever happened before; decisions that must be
        //      uniform (leave, merge) are taken by thread 0 alone and published through shared memory.
        // A piece of a split segment: who merges is settled by a ticket.  Thread 0 draws it as soon as its own last
        // tile is done -- the atomic's round trip then hides behind the rest of the piece -- and the CTA that draws
        // the last ticket of the segment is the merger: every other piece of the segment belongs to a CTA that has
        // drawn before it, hence is running and will deliver its partial without depending on anyone.  The merger
        // keeps its own part in registers, waits (bounded) for the others' delivery count, and combines.
        if (!prior_done) { wait_prior_launch(); prior_done = true; }  // (all 256 threads; returns at once when it has completed)
        const int seg_t0 = w.t - pc.tile0, seg_t1 = seg_t0 + pc.seg_nt;
        int c_first = cta, c_last = cta, n_pieces = 1, ticket = -1;  // (no ticket drawn: never the merger)
        int* seg_cnt = p.plan.seg_count + 2 * (pc.v * p.Hkv + pc.kvh);  // [0] tickets drawn, [1] partials delivered
        using St = Stage<D, MODE>;
        if (MODE != kTcCluster && !pc.complete) {
            segment_ctas(cs, p.n_ctas, cta, seg_t0, seg_t1, c_first, c_last);
            if (tid == 0 && !*abort) {
                n_pieces = segment_pieces(cs, c_first, c_last, seg_t0, seg_t1);
                ticket = atomicAdd(seg_cnt, 1);
            }
        }
        if (warp_active) {  // every P V of the piece has completed: the last one of each stream
            ok = ok && wait_all(&bars->pv_done[0], (w.u_base[0] + ((pc.nt + 1) >> 1) - 1) & 1, abort);
            if (pc.nt >= 2) ok = ok && wait_all(&bars->pv_done[1], (w.u_base[1] + (pc.nt >> 1) - 1) & 1, abort);
        }
        tc_fence_after();
        const bool two = pc.nt >= 2;
        // Stream exchange: group 1 hands its (m, l) to group 0, which answers with the two scale factors.
        // A thread only ever touches the two slots of its own row, so one barrier each way is enough.
        if (s == 1) { ex[r] = m; ex[kMaxRows + r] = l; }
        if (tid == 0) bars->epi_flag = (*abort ? 2 : 0) | ((MODE != kTcCluster && !pc.complete && ticket == n_pieces - 1) ? 1 : 0) | ((n_pieces - 1) << 8);
        named_bar_sync(1, 256);
        const bool leave = (bars->epi_flag & 2) != 0;
        const bool merger = (bars->epi_flag & 1) != 0;
        const bool stage_ok = merger && w.t + pc.nt == e_c && (bars->epi_flag >> 8) <= St::kMaxOthers;  // uniform: from shared memory
        float a0 = 0.f, a1 = 0.f, mm = -INFINITY, L = 0.f;
        if (s == 0) {
            const float m1 = two ? ex[r] : -INFINITY, l1 = ex[kMaxRows + r];
            mm = fmaxf(m, m1);
            a0 = (m == -INFINITY) ? 0.f : exp2f(m - mm);
            a1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - mm);
            L = a0 * l + (two ? a1 * l1 : 0.f);
            if (pc.complete) { const float inv = 1.f / L; a0 *= inv; a1 *= inv; }
            ex[r] = a0;
            ex[kMaxRows + r] = a1;
        }
        named_bar_sync(1, 256);
        if (s == 1) { a0 = ex[r]; a1 = ex[kMaxRows + r]; }
        constexpr int kChunks = D / 64;  // 32-column chunks per softmax group
        const bool do_read = !leave && warp_active;
        // the load warps of this CTA have seen every page id of the segment by now
        const bool zero_rows = pc.complete && sequence_flagged(p, pc.b);
        float o[kChunks][32];  // this thread's row, its group's half of the columns
#pragma unroll
        for (int ch = 0; ch < kChunks; ++ch) {
            const int col = s * (D / 2) + ch * 32;
            if (do_read) {
                uint32_t o0[32], o1[32];
                tmem_ld32(tmem + lane_base + col_o[0] + col, o0);
                if (two) tmem_ld32(tmem + lane_base + col_o[1] + col, o1);
                tc_wait_ld();
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    o[ch][k] = __uint_as_float(o0[k]) * a0;
                    if (two) o[ch][k] = fmaf(__uint_as_float(o1[k]), a1, o[ch][k]);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 32; ++k) o[ch][k] = 0.f;
            }
            if (ch == kChunks - 1) {
                tc_fence_before();
                mbar_arrive(&bars->o_free);           // O has been read: the next piece may overwrite it
            }
            if (MODE == kTcCluster) {
                // one cluster per segment: a row another CTA owns goes to this CTA's scratch block for that owner, a row
                // this CTA owns to its own block in the K ring, idle since the last MMA (consecutive rows of a block
                // are consecutive 16-byte words: the warp's stores coalesce, and spread over the banks)
                const int dest = r / exch.share;
                if (do_read && r < pc.rows) {
                    unsigned char* blk = dest != cl_rank ? exch.g_block(dest) : exch.land + (size_t)cl_rank * exch.block;
#pragma unroll
                    for (int k = 0; k < 32; k += 4)
                        *reinterpret_cast<float4*>(blk + Exchange<D>::o_off(exch.share, r % exch.share, (col + k) >> 2)) =
                            make_float4(o[ch][k], o[ch][k + 1], o[ch][k + 2], o[ch][k + 3]);
                }
            } else if (do_read && r < pc.rows) {
                if (pc.complete) {
                    __nv_bfloat16* dst = p.out + ((long long)(pc.row0 + i) * p.Hq + pc.kvh * p.G + r % p.G) * D + col;
                    if (zero_rows) {  // by assignment: what was computed from a stand-in page may be inf or NaN
#pragma unroll
                        for (int k = 0; k < 32; ++k) o[ch][k] = 0.f;
                    }
                    store_cols_bf16<32>(dst, o[ch], 1.f);
                } else if (!merger) {
                    float4* dst = partial_o4(p.part, D, pc.slot, col, r);
#pragma unroll
                    for (int k = 0; k < 32; k += 4) dst[(k >> 2) * kMaxRows] = make_float4(o[ch][k], o[ch][k + 1], o[ch][k + 2], o[ch][k + 3]);
                }
            }
        }
        if (MODE == kTcCluster) {
            const int dest = r / exch.share, rl = r % exch.share;
            // (m, l) of the row for its owner (which may be this CTA: then into its own shared memory); a row this CTA
            // could not compute (it is giving up) counts as "saw no key"; a CTA whose load warps met a page id outside
            // the pool says so with a negative l
            if (r < pc.rows && s == 0) {
                const float2 ml = !do_read ? make_float2(-INFINITY, 0.f) : make_float2(mm, bars->bad ? -1.f : L);
                unsigned char* blk = dest != cl_rank ? exch.g_block(dest) : exch.land + (size_t)cl_rank * exch.block;
                *reinterpret_cast<float2*>(blk + exch.ml_off(rl)) = ml;
            }
            cluster_sync_all();  // all 256 threads, whatever happened before; the other warps of the CTA wait in the kernel body
            cl_synced = true;
            // (the cluster barrier is a barrier of this CTA's threads as well: its own block in the K ring is complete)
            if (warp == 0) cluster_fetch<D>(p, exch, bars, cl_rank);
            if (wait_all(&bars->merge_bar, 0, abort) && !leave) cluster_reduce<D>(p, exch, cl_rank, pc.rows, pc.kvh, pc.row0);
        } else if (do_read && r < pc.rows && !pc.complete && s == 0) {
            // (the merger too: both column halves of its row need them, and only this thread has them)
            if (stage_ok) {
                float* own_ml = reinterpret_cast<float*>(stage + St::kMlOffset);
                own_ml[r] = mm;
                own_ml[kMaxRows + r] = L;
            } else {
                p.part.m[pc.slot * kMaxRows + r] = mm;
                p.part.l[pc.slot * kMaxRows + r] = L;
            }
        }
        if (MODE != kTcCluster && !pc.complete) {
            if (!merger) {
                // deliver: the barrier orders the partial stores of all threads before thread 0's fence, the fence
                // before the count.  Nobody waits for the count's result: the CTA goes straight on to its next piece.
                named_bar_sync(1, 256);
                if (tid == 0 && !leave && !*abort) {
                    __threadfence();
                    atomicAdd(seg_cnt + 1, 1);
                }
            } else {
                if (tid == 0) {
                    // the n - 1 other pieces: all drawn before ours, so their CTAs are past their last tile
                    const unsigned long long t_start = global_ns();
                    bool there = false;
                    for (uint32_t it = 0; !there; ++it) {
                        int v;
                        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(seg_cnt + 1) : "memory");
                        there = v >= n_pieces - 1;
                        if (!there && (it & 15u) == 15u && (*abort || global_ns() - t_start > kWaitLimitNs)) break;
                    }
                    if (there) {
                        seg_cnt[0] = 0;  // everyone has drawn and delivered: ready for the next call
                        seg_cnt[1] = 0;
                        bars->epi_flag |= 4;  // go: read after the barrier below, so that all 256 threads decide alike
                    } else {
                        *abort = 1;
                    }
                }
                // At the last piece of the range the Q tile and the K and V rings are idle (every load of this CTA has
                // been consumed): the other pieces (m, l, and the O arrays in rounds) are brought there by bulk copies, all
                // of a round in flight together, and the merge reads shared memory.  Read straight from L2 the merge is
                // a chain of dependent round trips (row maxima, then piece after piece), each 1-2 us while the other SMs
                // still stream: measured 7-9 us for two or three pieces.
                auto issue_round = [&](int round) {  // thread 0
                    const int k0 = round * St::kRound, k1 = min(n_pieces - 1, k0 + St::kRound);
                    mbar_arrive_expect_tx(&bars->merge_bar, (uint32_t)(k1 - k0) * St::kPieceBytes + (round == 0 ? (uint32_t)(n_pieces - 1) * 2 * kMaxRows * 4 : 0u));
                    int k = 0;
                    for (int c = c_first; c <= c_last; ++c) {
                        const int sc = cs.at(c), ec = cs.at(c + 1);
                        if (c == cta || max(sc, seg_t0) >= min(ec, seg_t1)) continue;
                        const int slot = 2 * c + (sc >= seg_t0 ? 0 : 1);
                        if (round == 0) {
                            unsigned char* mlk = stage + St::kMlOffset + (size_t)(1 + k) * 2 * kMaxRows * 4;
                            bulk_load(mlk, p.part.m + slot * kMaxRows, kMaxRows * 4, &bars->merge_bar);
                            bulk_load(mlk + kMaxRows * 4, p.part.l + slot * kMaxRows, kMaxRows * 4, &bars->merge_bar);
                        }
                        if (k >= k0 && k < k1)
                            bulk_load(stage + (size_t)(k - k0) * St::kPieceBytes, p.part.o + (size_t)slot * (St::kPieceBytes / 4), St::kPieceBytes,
                                      &bars->merge_bar);
                        ++k;
                    }
                };
                if (tid == 0 && (bars->epi_flag & 4) && stage_ok) {
                    fence_proxy_async_all();
                    issue_round(0);
                    int own_pos = 0;
                    for (int c = c_first; c < cta; ++c) own_pos += max(cs.at(c), seg_t0) < min(cs.at(c + 1), seg_t1);
                    // (after the acquire: every CTA of the segment has looked up its page ids by now)
                    bars->epi_flag |= (own_pos << 16) | (sequence_flagged(p, pc.b) ? 8 : 0);
                }
                named_bar_sync(1, 256);  // orders the acquire before every thread's loads of the partials
                const int rr = tid & (kMaxRows - 1), cg = tid >> 7;
                // rr == r and cg == s: the columns a thread merges are the ones it holds in registers
                if ((bars->epi_flag & 4) && !leave) {
                    if (!stage_ok) {
                        if (rr < pc.rows)
                            merge_row<D, D / 2>(p, cs, c_first, c_last, pc.b, pc.kvh, pc.row0, seg_t0, seg_t1, rr, cg, &o[0][0], cta);
                    } else {
                        merge_staged<D, MODE>(p, bars, stage, (int)((bars->epi_flag >> 8) & 0xff), (int)(bars->epi_flag >> 16), &o[0][0], rr, cg,
                                              rr < pc.rows, (bars->epi_flag & 8) != 0, pc.kvh, pc.row0, abort, issue_round);
                    }
                }
            }
        }
        if (leave) break;
        w.advance(pc);
    }
    // a CTA that gave up before its epilogue still owes the cluster its arrival: the peers must not wait for ever
    if (MODE == kTcCluster && !cl_synced) cluster_sync_all();
}

// ---------------------------------------------------------------------------------------------
// A call that plans for itself (kTcSelfPlanned, kTcCluster): at most kSelfPlanMaxRb sequences, one row block
// each.  Warp 0 of every CTA checks the lengths and makes the scans the plan kernel would have made, into
// shared memory; the roles then read them through the same Plan pointers.  No launch, no dependency.
// ---------------------------------------------------------------------------------------------
template <int MODE>
__device__ __forceinline__ void self_plan(const AttnParams& p, SelfScans* sc, RowBlock* rbs, int* s_cs, int* s_first) {
    const int lane = threadIdx.x & 31, B = p.batch;
    const bool live = lane < B;
    long long n = 0, Lq = 0, M = 0, nb = 1;
    bool bad = false;
    if (live) {
        n = p.prefix_lens[lane]; Lq = p.q_lens[lane]; M = p.n_mask[lane];
        nb = p.n_blocks ? p.n_blocks[lane] : 1;
        bad = n < 0 || Lq < 0 || M < 0 || M > Lq || Lq > p.max_q_len || n + Lq > (long long)p.max_pages * 16;
        bad = bad || nb < 0 || (nb > 1 && (M % nb != 0 || nb > Lq - M));  // equal mask blocks, one hypothesis each
        if (bad) Lq = 0;
    }
    int q = (int)Lq, t = Lq > 0 ? (int)((n + Lq + kTileTokens - 1) / kTileTokens) : 0, ne = t > 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int uq = __shfl_up_sync(0xffffffffu, q, o), ut = __shfl_up_sync(0xffffffffu, t, o), un = __shfl_up_sync(0xffffffffu, ne, o);
        if (lane >= o) { q += uq; t += ut; ne += un; }
    }
    const int rows = __shfl_sync(0xffffffffu, q, 31);
    const bool fatal = __any_sync(0xffffffffu, bad) || rows != p.total_q_rows;
    if (live) {
        sc->cu_q[lane + 1] = q; sc->cu_tiles[lane + 1] = t; sc->cu_ne[lane + 1] = ne;
        const RowBlock rb = {lane, 0, (int)n, (int)Lq, (int)M, (int)nb, {0, 0}};
        rbs[lane] = rb;
    }
    if (lane == 0) {
        sc->cu_q[0] = 0; sc->cu_tiles[0] = 0; sc->cu_ne[0] = 0;
        sc->fatal = fatal;
        if (fatal && blockIdx.x == 0) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
    }
    if (MODE == kTcSelfPlanned) {
        // the range starts of this CTA and its neighbours, a lane each: the cuts the plan kernel would have made
        // (range_cut is shared with it and with the host), all in one go instead of one after the other
        __syncwarp();
        const int tiles = __shfl_sync(0xffffffffu, t, 31), nonempty = __shfl_sync(0xffffffffu, ne, 31);
        const long long k = p.piece_cost, W = (long long)p.Hkv * (tiles + k * nonempty);
        const int total = fatal ? 0 : tiles * p.Hkv;
        const int n_use = ranges_in_use(W, k, p.min_range_tiles, p.n_ctas);
        const int cc = (int)blockIdx.x - kCsWindow / 2 + 1 + lane;
        int start = 0, first = 0;
        if (cc >= 0 && cc <= p.n_ctas) {
            const int* ct_ = sc->cu_tiles;
            const int* ne_ = sc->cu_ne;
            start = (cc >= n_use || total == 0) ? total
                                                : range_cut(cc, n_use, W, B, p.Hkv, k, [ct_](int b) { return ct_[b]; }, [ne_](int b) { return ne_[b]; }, &first);
        }
        s_cs[lane] = start;
        if (cc == (int)blockIdx.x) *s_first = first;
    }
}

template <int D, int MODE>
__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap qmap,
                                                              const AttnParams p_in) {
    using C = Cfg<D, MODE>;
    extern __shared__ __align__(1024) unsigned char smem[];  // the swizzled tiles need 1024-byte alignment
    unsigned char* sq = smem;
    unsigned char* sk = smem + C::kQBytes;                      // K ring
    unsigned char* sv = sk + C::kStages * C::kKBytes;           // V ring
    Bars* bars = reinterpret_cast<Bars*>(smem + C::kBarOffset);
    float* ex = reinterpret_cast<float*>(smem + C::kExOffset);
    int* s_cs = reinterpret_cast<int*>(smem + C::kCsOffset);
    Piece* ring = reinterpret_cast<Piece*>(smem + C::kDescOffset);
    SelfScans* scans = reinterpret_cast<SelfScans*>(smem + C::kScanOffset);
    RowBlock* rbs = reinterpret_cast<RowBlock*>(smem + C::kRbOffset);
    volatile int* abort = &bars->abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if ((smem_u32(smem) & 1023u) != 0u) {  // uniform; cannot happen with the declared alignment: leave before any barrier
        if (tid == 0) atomicOr(p_in.status, FD_DEV_TIMEOUT);
        return;
    }

    // ---- set-up that needs nothing from earlier kernels: under programmatic dependent launch it overlaps the
    //      tail of the previous launch on the stream (the plan kernel, or the previous layer's call);
    //      griddepcontrol.wait below is where that launch's results are needed
    if (warp == 1 && lane == 0) {
        for (int i = 0; i < C::kStages; ++i) {
            mbar_init(&bars->k_full[i], 1); mbar_init(&bars->k_empty[i], 1);
            mbar_init(&bars->v_full[i], 1); mbar_init(&bars->v_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->s_full[i], 1);
            mbar_init(&bars->p_full[i], 128);
            mbar_init(&bars->pv_done[i], 1);
        }
        mbar_init(&bars->q_full, 1);
        mbar_init(&bars->q_free, 1);
        mbar_init(&bars->o_free, 256);
        mbar_init(&bars->merge_bar, 1);
        bars->abort = 0;
        bars->epi_flag = 0;
        bars->desc_n = 0;
        bars->piece_ok = 0;
        bars->bad = 0;
        mbar_fence_init();
    }
    if (warp == kMmaWarp) tmem_alloc(&bars->tmem_base, 512);
    if (warp == kKWarp && lane == 0) { prefetch_tmap(&tmap); prefetch_tmap(&qmap); }
    // a call that plans for itself: warp 0 does so meanwhile (it needs the earlier kernels' results -- the lengths --
    // and waits for them on its own; its global loads then overlap the set-up of the other warps)
    if (MODE != kTcPlanned && warp == 0) {
        if (!p_in.early) wait_prior_launch();
        self_plan<MODE>(p_in, scans, rbs, s_cs, &bars->first);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    // a dependent launch behind this one (the next layer's call) may bring its CTAs in as ours retire and do its
    // own set-up; it waits for this grid to complete before reading anything
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Everything below the plan needs the results of the launch before this one.  Under a pinned plan that launch is
    // normally the previous layer's call (p.early): it writes neither the plan nor the lengths nor the page table, so
    // the work of this CTA, its first piece and its first page ids are looked up while it still runs -- three to five
    // dependent L2 round trips, 2.4 us -- and each role waits for it just before its first access to anything else.
    if (!p_in.early) wait_prior_launch();

    // ---- the work of this CTA
    AttnParams p = p_in;
    const int cta = blockIdx.x;
    int total, n_rb, fatal;
    Range rg = {0, 0, 0};
    CtaStarts cs = {};
    cs.s = s_cs;
    cs.base = cta - kCsWindow / 2 + 1;
    int cl_rank = 0, cl_rows = 0, cl_b = 0, cl_kvh = 0, cl_row0 = 0;  // kTcCluster: this CTA's place and its segment
    bool cl_idle = false;
    if (MODE == kTcPlanned) {
        const PlanHeader hdr = *p.plan.hdr;
        total = hdr.total_tiles; n_rb = hdr.n_rb; fatal = hdr.fatal;
        if (total) { rg.s_c = p.plan.cta_start[cta]; rg.e_c = p.plan.cta_start[cta + 1]; rg.first = p.plan.cta_first[cta]; }
        cs.g = p.plan.cta_start;
    } else {
        p.plan.rb = rbs; p.plan.cu_q = scans->cu_q; p.plan.cu_tiles = scans->cu_tiles; p.plan.cu_ne = scans->cu_ne;
        n_rb = p.batch;
        fatal = scans->fatal;
        const int tiles = scans->cu_tiles[n_rb], nonempty = scans->cu_ne[n_rb];
        total = fatal ? 0 : tiles * p.Hkv;
        if (MODE == kTcSelfPlanned) {
            // the ranges the plan kernel would have cut (range_cut is shared with it and with the host)
            cs.ct = scans->cu_tiles; cs.ne = scans->cu_ne;
            cs.n_rb = n_rb; cs.Hkv = p.Hkv; cs.k = p.piece_cost; cs.total = total;
            cs.W = (long long)p.Hkv * (tiles + (long long)p.piece_cost * nonempty);
            cs.n_use = ranges_in_use(cs.W, p.piece_cost, p.min_range_tiles, p.n_ctas);
            if (total) { rg.s_c = s_cs[cta - cs.base]; rg.e_c = s_cs[cta + 1 - cs.base]; rg.first = bars->first; }
        } else {
            // segment = cluster number; the cluster's CTAs take equal shares of its tiles, in rank order
            const int seg = cta / p.cluster, v = seg / p.Hkv;
            cl_rank = (int)cluster_ctarank();
            cl_kvh = seg % p.Hkv;
            cl_b = v;
            cl_rows = rbs[v].Lq * p.G;
            cl_row0 = scans->cu_q[v];
            const int T = total ? scans->cu_tiles[v + 1] - scans->cu_tiles[v] : 0;
            const int t_base = p.Hkv * scans->cu_tiles[v] + cl_kvh * T;
            // (T <= 2^23 tiles and at most 16 ranks: the products fit 32 bits)
            rg.s_c = t_base + (int)((unsigned)T * (unsigned)cl_rank / (unsigned)p.cluster);
            rg.e_c = t_base + (int)((unsigned)T * (unsigned)(cl_rank + 1) / (unsigned)p.cluster);
            rg.first = v;
            cl_idle = rg.s_c >= rg.e_c && T > 0;  // peers have tiles: stay for the merge
        }
    }
    // Reading q and the cache ahead of the launch before this one pays where a call is short (its start and the tail
    // of the call before it overlap); a CTA with a long range gains nothing and only takes bandwidth from the
    // stragglers of that call, which everyone then waits for (measured: + 1.5 % on 222 tiles per CTA).
    if (p.early >= 2 && rg.e_c - rg.s_c > kEarlyLoadMaxTiles) p.early = 1;
    if (rg.s_c >= rg.e_c && !cl_idle) {  // uniform (over the cluster too): no tile for this CTA, or nothing at all
        if (p.early) wait_prior_launch();
        if (total == 0 && fatal) {  // inconsistent lengths: a defined output, zeros
            const long long n16 = (long long)p.total_q_rows * p.Hq * D / 8;
            uint4* o = reinterpret_cast<uint4*>(p.out);
            for (long long i2 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i2 < n16; i2 += (long long)gridDim.x * blockDim.x)
                o[i2] = make_uint4(0, 0, 0, 0);
        }
        __syncthreads();
        if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
        return;
    }
    Exchange<D> exch = {};
    if (MODE == kTcCluster) {
        exch.g_base = reinterpret_cast<unsigned char*>(p.part.o) + (size_t)cta * 2 * kMaxRows * D * 4;
        exch.land = sk;
        exch.land_s = smem_u32(sk);
        exch.share = cluster_share(p.cluster);
        exch.block = cluster_block_bytes(p.cluster, D);
    }
    if (MODE == kTcCluster && cl_idle) {
        // fewer tiles than CTAs in the cluster: this one tells every owner "saw no key" and combines the rows it owns
        if (p.early) wait_prior_launch();
        if (tid < cl_rows) {
            const int dest = tid / exch.share, rl = tid % exch.share;
            unsigned char* blk = dest != cl_rank ? exch.g_block(dest) : exch.land + (size_t)cl_rank * exch.block;
            *reinterpret_cast<float2*>(blk + exch.ml_off(rl)) = make_float2(-INFINITY, 0.f);
        }
        cluster_sync_all();  // (a CTA-wide barrier as well: the own block is complete)
        if (warp == 0) cluster_fetch<D>(p, exch, bars, cl_rank);
        if (tid < 2 * kMaxRows) {  // whole warps: the wait is warp-uniform
            if (wait_all(&bars->merge_bar, 0, abort)) cluster_reduce<D>(p, exch, cl_rank, cl_rows, cl_kvh, cl_row0);
        }
    } else if (warp < 8) {
        // Warp-specialised register budgets: the softmax groups keep a whole 128-column row of S in registers.
        // 8 x 32 x 224 + 4 x 32 x 56 = 384 x 168, what the launch allocated: the increase is served exactly by what
        // the decrease released (a request for more than that does not return).
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        softmax_role<D, MODE>(p, bars, ex, s_cs, cs, ring, tmem, rg, exch, cl_rank, sq, sv, abort);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if (warp == kKWarp) load_role<D, MODE>(tmap, p, n_rb, sk, bars->k_full, bars->k_empty, 0, rg, &bars->k_full[0], &bars->bad, abort);
        else if (warp == kVWarp) load_role<D, MODE>(tmap, p, n_rb, sv, bars->v_full, bars->v_empty, 1, rg, &bars->k_full[0], &bars->bad, abort);
        else if (warp == kMmaWarp) mma_role<D, MODE>(p, sq, sk, sv, bars, ring, tmem, rg, abort);
        else q_role<D, MODE>(qmap, p, n_rb, sq, bars, ring, rg, abort);
        if (MODE == kTcCluster) cluster_sync_all();  // the cluster barrier of the merge counts every thread
    }
    // ---- common tail: everything of this CTA has completed, or it is giving up
    if (*abort && tid == 0) atomicOr(p.status, FD_DEV_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
}

struct TmapEntry {
    const void* ptr;
    int n;  // KV pool: pages; q: rows
    CUtensorMap map;
};

// Tensor maps already encoded, keyed by (pointer, extent).  A model calls the attention once per layer with that
// layer's pool and q buffer, in the same order every step: the entry after the last hit is tried first, then the
// whole list; the list grows with the number of distinct operands (one per layer) and is recycled round-robin
// only past kMaxEntries.
struct TmapCache {
    static constexpr size_t kMaxEntries = 4096;
    std::vector<TmapEntry> e;
    size_t last = 0, victim = 0;
    const CUtensorMap* find(const void* ptr, int n) {
        const size_t cnt = e.size();
        for (size_t k = 0; k < cnt; ++k) {
            const size_t i = (last + 1 + k) % cnt;
            if (e[i].ptr == ptr && e[i].n == n) { last = i; return &e[i].map; }
        }
        return nullptr;
    }
    TmapEntry& slot() {
        if (e.size() < kMaxEntries) { e.emplace_back(); last = e.size() - 1; return e.back(); }
        last = victim;
        victim = (victim + 1) % kMaxEntries;
        return e[last];
    }
};

struct TcState {
    PFN_cuTensorMapEncodeTiled_v12000 encode;
    TmapCache kv, q;
    int d, hkv;
    const CUtensorMap* current;
    const CUtensorMap* qcurrent;
    int max_clusters[kMaxCluster + 1];  // [C]: clusters of C CTAs of the cluster kernel the device holds at once (0 = not launchable)
};

template <int D, int MODE>
cudaError_t configure_kernel() {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<D, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D, MODE>::kSmemBytes);
    if (e == cudaSuccess && MODE == kTcCluster)
        e = cudaFuncSetAttribute(attn_tc_kernel<D, MODE>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    return e;
}

// How many clusters of `c` CTAs of the cluster kernel can be resident together (0 if such a launch is refused).
template <int D>
int query_clusters(int c, int n_sms) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((n_sms / c) * c);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Cfg<D, kTcCluster>::kSmemBytes;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<D, kTcCluster>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

template <int D, int MODE>
void launch_mode(const TcState* st, const AttnParams& p, cudaStream_t s) {
    // Programmatic dependent launch: the CTAs may start while the previous launch on the stream (the plan kernel,
    // or the previous layer's call) is still running; they do their set-up and then wait for it inside the kernel.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.dynamicSmemBytes = Cfg<D, MODE>::kSmemBytes;
    if (MODE == kTcCluster) {
        cfg.gridDim = dim3(p.batch * p.Hkv * p.cluster);  // one cluster per (sequence, kv-head) segment
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = p.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    cudaLaunchKernelEx(&cfg, attn_tc_kernel<D, MODE>, *st->current, *st->qcurrent, p);
}

}  // namespace

bool attn_tc_supported(int d, int G, int max_q_len) {
    (void)max_q_len;  // any length: a long query block is cut into row blocks of kMaxRows / G block rows
    return (d == 64 || d == 128) && G <= kMaxRows;
}

// Looks up (or encodes) the tensor map of this KV pool: a 4-D view [groups of 8 rows][d / 64 halves][8 rows][64]
// with a box of one page of one kv-head (two groups, both halves) and 128-byte swizzle.
cudaError_t attn_tc_prepare(void** state, const AttnParams& p) {
    TcState* st = static_cast<TcState*>(*state);
    if (!st) {
        st = new TcState();
        st->encode = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", reinterpret_cast<void**>(&st->encode), cudaEnableDefault, &qres);
        if (e != cudaSuccess || !st->encode) { delete st; return e != cudaSuccess ? e : cudaErrorNotSupported; }
        st->d = p.d; st->hkv = p.Hkv;
        if (p.d == 64) {
            e = configure_kernel<64, kTcPlanned>();
            if (e == cudaSuccess) e = configure_kernel<64, kTcSelfPlanned>();
            if (e == cudaSuccess) e = configure_kernel<64, kTcCluster>();
        } else {
            e = configure_kernel<128, kTcPlanned>();
            if (e == cudaSuccess) e = configure_kernel<128, kTcSelfPlanned>();
            if (e == cudaSuccess) e = configure_kernel<128, kTcCluster>();
        }
        if (e != cudaSuccess) { delete st; return e; }
        int n_sms = 0, dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
        for (int c = 0; c <= kMaxCluster; ++c) st->max_clusters[c] = 0;
        for (int c = 2; c <= kMaxCluster; ++c) {
            const bool fits = cluster_fits(c, p.d);
            st->max_clusters[c] = !fits ? 0 : p.d == 64 ? query_clusters<64>(c, n_sms) : query_clusters<128>(c, n_sms);
        }
        *state = st;
    }
    // q: a 3-D view [T][Hq][d], box = 64 elements x G q-heads (one kv-head) x q_box_t block rows
    st->qcurrent = st->q.find(p.q, p.total_q_rows);
    if (!st->qcurrent) {
        CUtensorMap map;
        cuuint64_t dims[3] = {(cuuint64_t)p.d, (cuuint64_t)p.Hq, (cuuint64_t)(p.total_q_rows > 0 ? p.total_q_rows : 1)};
        cuuint64_t strides[2] = {(cuuint64_t)p.d * 2, (cuuint64_t)p.Hq * p.d * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)p.G, (cuuint32_t)p.q_box_t};
        cuuint32_t estr[3] = {1, 1, 1};
        const CUresult r = st->encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(p.q), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
        TmapEntry& e = st->q.slot();
        e.ptr = p.q;
        e.n = p.total_q_rows;
        e.map = map;
        st->qcurrent = &e.map;
    }
    st->current = st->kv.find(p.kv, p.num_pages);
    if (st->current) return cudaSuccess;
    // 64 elements x 8 rows x the 64-wide halves of d x groups of 8 rows: a box of two groups is one page of one
    // kv-head and lands as [group][half][8 rows][128 B]
    CUtensorMap map;
    cuuint64_t dims[4] = {64, 8, (cuuint64_t)p.d / 64, (cuuint64_t)p.num_pages * 2 * p.Hkv * 2};
    cuuint64_t strides[3] = {(cuuint64_t)p.d * 2, 128, (cuuint64_t)p.d * 2 * 8};
    cuuint32_t box[4] = {64, 8, (cuuint32_t)p.d / 64, 2};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = st->encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(p.kv), dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    TmapEntry& e = st->kv.slot();
    e.ptr = p.kv;
    e.n = p.num_pages;
    e.map = map;
    st->current = &e.map;
    return cudaSuccess;
}

// CTAs per cluster for a call with one cluster per segment: the largest size (any, not only powers of two: a GPC holds
// a limited number of clusters of each size) for which all clusters of the call are resident together, so every SM it
// can use streams at once and a CTA has the fewest tiles; 0 if there is none.
int attn_tc_cluster_size(const void* state, int n_segments, int n_sms) {
    const TcState* st = static_cast<const TcState*>(state);
    if (!st || n_segments <= 0) return 0;
    for (int c = kMaxCluster; c >= 2; --c)
        if (n_segments * c <= n_sms && st->max_clusters[c] >= n_segments) return c;
    return 0;
}

void launch_attn_tc(void* state, const AttnParams& p, int mode, cudaStream_t s) {
    if (p.batch == 0) return;
    const TcState* st = static_cast<const TcState*>(state);
    if (p.d == 64) {
        if (mode == kTcCluster) launch_mode<64, kTcCluster>(st, p, s);
        else if (mode == kTcSelfPlanned) launch_mode<64, kTcSelfPlanned>(st, p, s);
        else launch_mode<64, kTcPlanned>(st, p, s);
    } else {
        if (mode == kTcCluster) launch_mode<128, kTcCluster>(st, p, s);
        else if (mode == kTcSelfPlanned) launch_mode<128, kTcSelfPlanned>(st, p, s);
        else launch_mode<128, kTcPlanned>(st, p, s);
    }
}

void attn_tc_free(void* state) { delete static_cast<TcState*>(state); }

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing will ever arrive on.
// The wait gives up after `limit_ns`, the kernel raises FD_DEV_TIMEOUT and returns normally.
__global__ void wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; mbar_fence_init(); }
    __syncthreads();
    const bool ok = mbar_wait_ns(&bar, 0, &abort_flag, limit_ns);
    __syncwarp();
    if (threadIdx.x == 0 && !ok) atomicOr(status, FD_DEV_TIMEOUT);
}

void launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, cudaStream_t s) {
    wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status, limit_ns);
}

}  // namespace fd
