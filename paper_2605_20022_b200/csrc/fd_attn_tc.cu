// Tensor-core split-KV attention under the hybrid mask for sm_100a: TMA-staged KV pages,
// tcgen05 MMAs with accumulators in tensor memory, softmax in registers.
//
// Work decomposition.  The plan kernel numbers all 128-token KV tiles of the call
// (sequence-major, then kv-head, then position) and each of the n_ctas persistent CTAs takes
// one contiguous range, so every SM streams the same number of KV bytes.  A range is walked
// piece by piece, a piece being its intersection with one (sequence b, kv-head) segment.
//
// One piece.  The G * Lq_b <= 128 query rows that share the kv-head (row r = block row
// r / G of q-head kvh * G + r % G) form the M = 128 operand of every MMA, so each KV tile is
// read from HBM once for all of them.  Per tile j of the piece:
//     producer warps: one for K, one for V; 16 lanes issue one 2 KB TMA box each (8 pages x two
//                     64-wide halves of d) into a 128B-swizzled buffer of a 3-deep ring per
//                     operand; a K buffer is released by the QK^T commit, a V buffer by P V;
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
// Every wait is bounded.  A wait that runs out raises a CTA-wide abort flag: all roles leave
// their loops, in-flight TMA copies are drained, TMEM is released and FD_DEV_TIMEOUT is set.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "fd_internal.cuh"
#include "fd_sm100.cuh"

namespace fd {

using namespace sm100;

namespace {

constexpr int kThreads = 384;  // warps 0-3 softmax group 0, 4-7 softmax group 1, 8 K loads, 9 V loads, 10 MMA, 11 idle
constexpr int kKWarp = 8, kVWarp = 9, kMmaWarp = 10;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct Cfg {
    static constexpr int kStages = (D == 128) ? 3 : 6;   // buffers in the K ring, and again in the V ring
    static constexpr int kQBytes = kMaxRows * D * 2;
    static constexpr int kKBytes = kTileTokens * D * 2;  // one K (or V) tile
    static constexpr int kBarOffset = kQBytes + 2 * kStages * kKBytes;
    static constexpr int kSmemBytes = kBarOffset + 512 + 1024;  // + barriers + slack for 1024-byte alignment
    static constexpr int kKSteps = D / 16;
    static constexpr int kHalves = D / 64;
};

struct Bars {
    uint64_t k_full[6], k_empty[6], v_full[6], v_empty[6];
    uint64_t s_full[2], p_full[2], pv_done[2];
    uint64_t all_done;
    uint32_t tmem_base;
    int abort;
    int merge_flag;
};

struct Piece {
    int b, kvh, tile0, nt, n, Lq, M, kv_len, rows, row0, slot;
    bool complete;
};

__device__ __forceinline__ Piece decode_piece(const AttnParams& p, int t, int s_c, int e_c, int cta) {
    Piece pc;
    int lo = 0, hi = p.batch;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (p.Hkv * p.plan.cu_tiles[mid] <= t) lo = mid; else hi = mid;
    }
    pc.b = lo;
    const int ntiles = p.plan.cu_tiles[lo + 1] - p.plan.cu_tiles[lo];
    const int rem = t - p.Hkv * p.plan.cu_tiles[lo];
    pc.kvh = rem / ntiles;
    pc.tile0 = rem % ntiles;
    const int seg_start = t - pc.tile0, seg_end = seg_start + ntiles;
    const int t_end = min(e_c, seg_end);
    pc.nt = t_end - t;
    pc.n = p.prefix_lens[lo];
    pc.Lq = p.q_lens[lo];
    pc.M = p.n_mask[lo];
    pc.kv_len = pc.n + pc.Lq;
    pc.rows = pc.Lq * p.G;
    pc.row0 = p.plan.cu_q[lo];
    pc.complete = (t == seg_start) && (t_end == seg_end);
    pc.slot = 2 * cta + (t == s_c ? 0 : 1);
    return pc;
}

#ifdef FD_TRACE
// Debug build only: per-role timestamps of CTA 0 for pipeline analysis.  Each role's tracing thread
// owns a region and a private counter, so an event costs one clock read and one store.
constexpr int kTraceRoles = 6, kTracePerRole = 4096;
__device__ unsigned long long g_trace[kTraceRoles * kTracePerRole];
__device__ unsigned int g_trace_n[kTraceRoles];
__device__ __forceinline__ void trace(int role, int ev, int tile, int& n) {
    if (blockIdx.x != 0 || n >= kTracePerRole) return;
    g_trace[role * kTracePerRole + n] = ((unsigned long long)clock64() & 0xffffffffffull) | ((unsigned long long)ev << 40) | ((unsigned long long)tile << 48);
    g_trace_n[role] = ++n;
}
#define TRACE(role, ev, tile) trace(role, ev, tile, tr_n)
#define TRACE_DECL int tr_n = 0
#else
#define TRACE(role, ev, tile)
#define TRACE_DECL
#endif

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Warp-uniform bounded wait.
__device__ __forceinline__ bool wait_all(uint64_t* bar, uint32_t parity, volatile int* abort) {
    const bool ok = mbar_wait(bar, parity, abort);
    return __all_sync(0xffffffffu, ok);
}

// Everything after the set-up, for one role class.  The two instantiations (softmax groups /
// producer + MMA warps) run in disjoint branches of the kernel so that each is compiled for its
// own register budget (setmaxnreg); they meet only at the CTA-wide barriers, which both execute
// the same number of times.
template <int D, bool kSoftmax>
__device__ __forceinline__ void run_role(const CUtensorMap& tmap, const AttnParams& p, unsigned char* sq, unsigned char* sk,
                                         unsigned char* sv, Bars* bars, int total, int s_c, int e_c) {
    using C = Cfg<D>;
    TRACE_DECL;
    float* ex_m = reinterpret_cast<float*>(sq);          // [2][128], aliases Q after the last MMA of a piece
    float* ex_l = ex_m + 2 * kMaxRows;
    volatile int* abort = &bars->abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const uint32_t tmem = bars->tmem_base;
    const uint32_t col_s[2] = {0u, 128u};
    const uint32_t col_o[2] = {256u, 384u};

    int g0 = 0;            // KV tiles this CTA has pushed through the stage ring so far
    int u_base[2] = {0, 0};  // tiles each stream has processed so far
    int piece_idx = 0;
    int issued = 0;        // producer: tiles whose loads were issued

    // The two load warps never take part in the per-piece barriers: they walk the pieces on their own,
    // held back only by the K / V rings, so the rings are already full when the MMAs of the next piece start.
    const bool loader = !kSoftmax && (warp == kKWarp || warp == kVWarp);
    const int ltid = warp < 8 ? tid : tid - 64;                 // index among the kPieceThreads other threads
    constexpr int kPieceThreads = kThreads - 64;

    for (int t = s_c; t < e_c;) {
        const Piece pc = decode_piece(p, t, s_c, e_c, cta);
        if (tid == 0) TRACE(5, 2, piece_idx);

        // ---- Q tile -> shared memory, K-major, 128-byte swizzle; rows beyond the block are zero
        if (!loader) {
            constexpr int kChunks = kMaxRows * (D / 8);                               // 16-byte chunks of the tile
            constexpr int kIters = (kChunks + kPieceThreads - 1) / kPieceThreads;
            uint4 v[kIters];
#pragma unroll
            for (int it = 0; it < kIters; ++it) {                                     // all loads in flight first
                const int idx = ltid + it * kPieceThreads, r = idx / (D / 8), ch = idx % (D / 8);
                v[it] = make_uint4(0, 0, 0, 0);
                if (idx < kChunks && r < pc.rows)
                    v[it] = *reinterpret_cast<const uint4*>(p.q + ((long long)(pc.row0 + r / p.G) * p.Hq + pc.kvh * p.G + r % p.G) * D + ch * 8);
            }
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int idx = ltid + it * kPieceThreads, r = idx / (D / 8), ch = idx % (D / 8);
                const int half = ch >> 3, c16 = ch & 7;
                if (idx < kChunks)
                    *reinterpret_cast<uint4*>(sq + half * (kMaxRows * 128) + r * 128 + ((c16 ^ (r & 7)) << 4)) = v[it];
            }
        }
        if (!loader) {
            fence_proxy_async_smem();
            named_bar_sync(2, kPieceThreads);
            if (tid == 0) TRACE(5, 3, piece_idx);
        }

        if constexpr (!kSoftmax) {
        if (warp == kKWarp || warp == kVWarp) {
            // ============================== TMA producers ==============================
            // K and V travel through separate rings: a K buffer is free again as soon as QK^T of its
            // tile has completed, a V buffer once P V has, so loads run several tiles ahead of the MMAs.
            const int which = (warp == kVWarp) ? 1 : 0;
            unsigned char* ring = which ? sv : sk;
            uint64_t* full = which ? bars->v_full : bars->k_full;
            uint64_t* empty = which ? bars->v_empty : bars->k_empty;
            constexpr int kOps = 8 * C::kHalves;
            const int pg = lane / C::kHalves, half = lane % C::kHalves;
            const int32_t* table = p.page_table + (long long)pc.b * p.max_pages;
            // the page id of the next tile is fetched before waiting for a free buffer, so the
            // table lookup never sits between a buffer becoming free and its refill
            auto page_of = [&](int j) -> int {
                const int pos = (pc.tile0 + j) * kTileTokens + pg * 16;
                if (!(j < pc.nt && lane < kOps && pos < pc.kv_len)) return -1;
                int id = table[pos >> 4];
                if ((unsigned)id >= (unsigned)p.num_pages) {  // never form an address from a bad id
                    p.plan.seq_ok[pc.b] = 0;
                    atomicOr(p.status, FD_DEV_BAD_PAGE);
                    id = 0;
                }
                return id;
            };
            int phys = page_of(0);
            for (int j = 0; j < pc.nt; ++j) {
                const int g = g0 + j, st = g % C::kStages, use = g / C::kStages;
                const int phys_next = page_of(j + 1);
                if (!wait_all(&empty[st], (use & 1) ^ 1, abort)) break;
                if (lane == 0) TRACE(which, 0, g0 + j);
                const int pos0 = (pc.tile0 + j) * kTileTokens;
                const int npg = min(8, (pc.kv_len - pos0 + 15) >> 4);
                if (lane == 0) mbar_arrive_expect_tx(&full[st], npg * (16 * D * 2));
                __syncwarp();
                if (phys >= 0) {
                    unsigned char* dst = ring + st * C::kKBytes + half * (kTileTokens * 128) + pg * 2048;
                    tma_load_2d(dst, &tmap, half * 64, ((phys * 2 + which) * p.Hkv + pc.kvh) * 16, &full[st]);
                }
                phys = phys_next;
                issued = g + 1;
            }
        } else if (warp == kMmaWarp) {
            // ============================== MMA issuer ==============================
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, kTileTokens, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, true);
            const uint32_t q_addr = smem_u32(sq);
            bool ok = true;
            auto issue_pv = [&](int jj) {
                const int gg = g0 + jj, s = jj & 1, st = gg % C::kStages, u = u_base[s] + (jj >> 1);
                if (!wait_all(&bars->v_full[st], (gg / C::kStages) & 1, abort)) { ok = false; return; }
                unsigned char* vt = sv + st * C::kKBytes;
                const int valid = pc.kv_len - (pc.tile0 + jj) * kTileTokens;
                if (valid < kTileTokens) {
                    // V rows no token owns may hold NaN or stale data: P is 0 there, but 0 * NaN is not
                    const int nbad = kTileTokens - valid;
                    for (int e = lane; e < nbad * 8 * C::kHalves; e += 32) {
                        const int r = valid + e / (8 * C::kHalves), w = e % (8 * C::kHalves);
                        *reinterpret_cast<uint4*>(vt + (w >> 3) * (kTileTokens * 128) + r * 128 + ((w & 7) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                if (!wait_all(&bars->p_full[s], u & 1, abort)) { ok = false; return; }
                tc_fence_after();
                if (lane == 0) {
                    TRACE(2, 2, g0 + jj);
                    const uint32_t v_addr = smem_u32(vt);
#pragma unroll
                    for (int kk = 0; kk < kTileTokens / 16; ++kk)
                        umma_ts(tmem + col_o[s], tmem + col_s[s] + kk * 8,
                                make_smem_desc(v_addr + kk * 2048, kTileTokens * 128, 1024), idesc_pv, jj >= 2 || kk > 0);
                    umma_commit(&bars->v_empty[st]);
                    umma_commit(&bars->pv_done[s]);
                }
                __syncwarp();
            };
            for (int j = 0; j < pc.nt && ok; ++j) {
                const int g = g0 + j, st = g % C::kStages, use = g / C::kStages;
                const int s = j & 1, u = u_base[s] + (j >> 1);
                if (!wait_all(&bars->k_full[st], use & 1, abort)) { ok = false; break; }
                if (lane == 0) TRACE(2, 0, g);
                if (u >= 1 && !wait_all(&bars->pv_done[s], (u - 1) & 1, abort)) { ok = false; break; }
                tc_fence_after();
                if (lane == 0) {
                    TRACE(2, 1, g);
                    const uint32_t k_addr = smem_u32(sk + st * C::kKBytes);
#pragma unroll
                    for (int kk = 0; kk < C::kKSteps; ++kk) {
                        const uint32_t off = (kk >> 2) * (kMaxRows * 128) + (kk & 3) * 32;
                        umma_ss(tmem + col_s[s], make_smem_desc(q_addr + off, 16, 1024), make_smem_desc(k_addr + off, 16, 1024),
                                idesc_qk, kk > 0);
                    }
                    umma_commit(&bars->k_empty[st]);
                    umma_commit(&bars->s_full[s]);
                }
                __syncwarp();
                if (j >= 1) issue_pv(j - 1);
            }
            if (ok) issue_pv(pc.nt - 1);
            if (ok && lane == 0) umma_commit(&bars->all_done);
            __syncwarp();
        }
        } else {
            // ============================== softmax groups ==============================
            const int s = warp >> 2;                  // stream
            const int r = (warp & 3) * 32 + lane;     // query row == TMEM lane
            const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
            const bool warp_active = (warp & 3) * 32 < pc.rows;
            const int i = r / p.G;
            const int limit = (r < pc.rows) ? ((i < pc.Lq - pc.M) ? pc.n + i + 1 : pc.kv_len) : 0;
            const float c = p.scale_log2e;
            float m = -INFINITY, l = 0.f;
            bool ok = true;

            // Warps whose 32 rows are all padding do nothing per tile: warp 0 of the group (always active)
            // arrives on p_full for them, and they wait at the epilogue's hardware barrier, not by polling.
            const int n_idle_threads = 32 * (4 - min(4, (pc.rows + 31) >> 5));
            for (int j = s; j < pc.nt && warp_active; j += 2) {
                const int u = u_base[s] + (j >> 1);
                if (!wait_all(&bars->s_full[s], u & 1, abort)) { ok = false; break; }
                tc_fence_after();
                if ((warp & 3) == 0 && lane == 0) TRACE(3 + s, 0, g0 + j);
                if (warp_active) {
                    const int pos0 = (pc.tile0 + j) * kTileTokens;
                    // tile reaches into the query block (or past kv_len): columns >= lim are invisible
                    const bool masked = pos0 + kTileTokens > pc.n;
                    const int lim = limit - pos0;
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
                                if (ch * 32 + k >= lim) sv[ch][k] = 0xff800000u;  // -inf by select: S may be NaN there
                    }
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
#pragma unroll
                        for (int k = 0; k < 32; k += 4) {
                            mx[0] = fmaxf(mx[0], __uint_as_float(sv[ch][k]));
                            mx[1] = fmaxf(mx[1], __uint_as_float(sv[ch][k + 1]));
                            mx[2] = fmaxf(mx[2], __uint_as_float(sv[ch][k + 2]));
                            mx[3] = fmaxf(mx[3], __uint_as_float(sv[ch][k + 3]));
                        }
                    const float m_new = fmaxf(m, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c);
                    if ((warp & 3) == 0 && lane == 0) TRACE(3 + s, 1, g0 + j);
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
                        asm volatile("" ::: "memory");    // keep the second half's math after this store (register pressure)
                    }
                    l += (sum0.x + sum0.y) + (sum1.x + sum1.y);
                    tc_wait_st();
                }
                tc_fence_before();
                mbar_arrive(&bars->p_full[s]);
                if ((warp & 3) == 0 && lane == 0 && n_idle_threads) mbar_arrive_cnt(&bars->p_full[s], n_idle_threads);
                if ((warp & 3) == 0 && lane == 0) TRACE(3 + s, 2, g0 + j);
            }

            // ---- epilogue: merge the two streams, then final rows, or a partial plus -- if this CTA is the
            //      last one to deliver a piece of the segment -- the merge of all its partials
            if (warp_active) ok = ok && wait_all(&bars->all_done, piece_idx & 1, abort);
            tc_fence_after();
            if (tid == 0) TRACE(5, 4, piece_idx);
            if (ok && warp_active) {  // (idle warps have not waited for the MMAs: Q, which this aliases, may still be read)
                ex_m[s * kMaxRows + r] = m;
                ex_l[s * kMaxRows + r] = l;
            }
            named_bar_sync(1, 256);
            if (ok && !*abort && warp_active) {
                const bool two = pc.nt >= 2;
                const float m0 = ex_m[r], m1 = two ? ex_m[kMaxRows + r] : -INFINITY;
                const float mm = fmaxf(m0, m1);
                const float a0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - mm);
                const float a1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - mm);
                const float L = a0 * ex_l[r] + (two ? a1 * ex_l[kMaxRows + r] : 0.f);
                const float inv = pc.complete ? 1.f / L : 1.f;
                constexpr int kChunks = D / 64;  // 32-column chunks per softmax group
#pragma unroll
                for (int ch = 0; ch < kChunks; ++ch) {
                    const int col = s * (D / 2) + ch * 32;
                    uint32_t o0[32], o1[32];
                    tmem_ld32(tmem + lane_base + col_o[0] + col, o0);
                    if (two) tmem_ld32(tmem + lane_base + col_o[1] + col, o1);
                    tc_wait_ld();
                    float o[32];
#pragma unroll
                    for (int k = 0; k < 32; ++k) {
                        o[k] = __uint_as_float(o0[k]) * a0;
                        if (two) o[k] = fmaf(__uint_as_float(o1[k]), a1, o[k]);
                        o[k] *= inv;
                    }
                    if (r < pc.rows) {
                        if (pc.complete) {
                            // the load warps of this CTA have seen every page id of the segment by now
                            if (!__ldcg(p.plan.seq_ok + pc.b)) {
#pragma unroll
                                for (int k = 0; k < 32; ++k) o[k] = 0.f;
                            }
                            __nv_bfloat16* dst = p.out + ((long long)(pc.row0 + i) * p.Hq + pc.kvh * p.G + r % p.G) * D + col;
#pragma unroll
                            for (int k = 0; k < 32; k += 8) {
                                __align__(16) __nv_bfloat162 v[4];
#pragma unroll
                                for (int q2 = 0; q2 < 4; ++q2) v[q2] = __floats2bfloat162_rn(o[k + 2 * q2], o[k + 2 * q2 + 1]);
                                *reinterpret_cast<uint4*>(dst + k) = *reinterpret_cast<const uint4*>(v);
                            }
                        } else {
                            float* dst = p.part.o + ((long long)pc.slot * D + col) * kMaxRows + r;
#pragma unroll
                            for (int k = 0; k < 32; ++k) dst[k * kMaxRows] = o[k];
                        }
                    }
                }
                if (!pc.complete && s == 0 && r < pc.rows) {
                    p.part.m[pc.slot * kMaxRows + r] = mm;
                    p.part.l[pc.slot * kMaxRows + r] = L;
                }
            }
            if (!pc.complete) {
                // Fused split merge: count the delivered pieces of the segment; whoever delivers the last
                // one combines them all (no CTA ever waits for another).  Both barriers are taken by all
                // 256 softmax threads whatever happened before, and thread 0 alone takes the decision.
                __threadfence();
                named_bar_sync(1, 256);
                if (tid == 0) {
                    int last = 0;
                    if (!*abort) {
                        const int ntiles = p.plan.cu_tiles[pc.b + 1] - p.plan.cu_tiles[pc.b];
                        const int seg_start = t - pc.tile0;
                        const int n = segment_pieces(seg_start, seg_start + ntiles, total, p.n_ctas);
                        last = atomicAdd(p.plan.seg_count + pc.b * p.Hkv + pc.kvh, 1) + 1 == n;
                    }
                    bars->merge_flag = last;
                }
                named_bar_sync(1, 256);
                if (bars->merge_flag) {
                    __threadfence();
                    const int rr = tid & (kMaxRows - 1), cg = tid >> 7;
                    if (rr < pc.rows) merge_row<D, D / 2>(p, total, pc.b, pc.kvh, rr, cg);
                }
            }
            tc_fence_before();
        }

        // ---- end of piece: every MMA and every epilogue read of this piece has completed (or the CTA is aborting)
        if (tid == 0) TRACE(5, 5, piece_idx);
        if (!loader) named_bar_sync(2, kPieceThreads);
        if (*abort) break;
        g0 += pc.nt;
        u_base[0] += (pc.nt + 1) >> 1;
        u_base[1] += pc.nt >> 1;
        ++piece_idx;
        t += pc.nt;
    }

    if (*abort) {
        // drain TMA copies still in flight before the shared memory is given back
        if (warp == kKWarp || warp == kVWarp) {
            uint64_t* full = (warp == kVWarp) ? bars->v_full : bars->k_full;
            for (int g = max(0, issued - C::kStages); g < issued; ++g) {
                const int st = g % C::kStages, use = g / C::kStages;
                const unsigned long long t0 = global_ns();
                for (uint32_t it = 0; it < kSpinLimit && global_ns() - t0 < kWaitLimitNs; ++it)
                    if (mbar_try_wait(&full[st], use & 1)) break;
            }
        }
        if (tid == 0) atomicOr(p.status, FD_DEV_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap tmap, AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sq = smem;
    unsigned char* sk = smem + C::kQBytes;                      // K ring
    unsigned char* sv = sk + C::kStages * C::kKBytes;           // V ring
    Bars* bars = reinterpret_cast<Bars*>(smem + C::kBarOffset);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const PlanHeader hdr = *p.plan.hdr;
    const int total = hdr.total_tiles;
    if (total == 0) {  // uniform: nothing allocated yet
        if (hdr.fatal) {  // inconsistent lengths: a defined output, zeros
            const long long n16 = (long long)p.total_q_rows * p.Hq * D / 8;
            uint4* o = reinterpret_cast<uint4*>(p.out);
            for (long long i2 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i2 < n16; i2 += (long long)gridDim.x * blockDim.x)
                o[i2] = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    const int cta = blockIdx.x;
    const int s_c = range_begin(cta, total, p.n_ctas), e_c = range_begin(cta + 1, total, p.n_ctas);
    if (s_c >= e_c) return;

    if (tid == 0) {
        for (int i = 0; i < C::kStages; ++i) {
            mbar_init(&bars->k_full[i], 1); mbar_init(&bars->k_empty[i], 1);
            mbar_init(&bars->v_full[i], 1); mbar_init(&bars->v_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->s_full[i], 1);
            mbar_init(&bars->p_full[i], 128);
            mbar_init(&bars->pv_done[i], 1);
        }
        mbar_init(&bars->all_done, 1);
        bars->abort = 0;
        mbar_fence_init();
    }
    if (warp == kMmaWarp) tmem_alloc(&bars->tmem_base, 512);
    if (warp == kKWarp && lane == 0) prefetch_tmap(&tmap);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // warp-specialised register budgets: the softmax groups keep a whole 128-column row of S in registers.
    // 8 x 32 x 216 + 4 x 32 x 72 = 384 x 168: exactly what the launch allocated, so the increase can
    // always be served by what the decrease released (asking for more than that never returns).
    if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        run_role<D, true>(tmap, p, sq, sk, sv, bars, total, s_c, e_c);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
        run_role<D, false>(tmap, p, sq, sk, sv, bars, total, s_c, e_c);
    }
}

struct TmapEntry {
    const void* ptr;
    int num_pages;
    CUtensorMap map;
};

struct TcState {
    PFN_cuTensorMapEncodeTiled_v12000 encode;
    TmapEntry cache[64];
    int n_cached, next;
    int d, hkv;
    const CUtensorMap* current;
};

}  // namespace

bool attn_tc_supported(int d, int G, int max_q_len) {
    return (d == 64 || d == 128) && G * max_q_len <= kMaxRows;
}

// Looks up (or encodes) the tensor map of this KV pool: a 2-D view [rows = pages*2*Hkv*16, d]
// with a 16-row x 64-element box and 128-byte swizzle.
cudaError_t attn_tc_prepare(void** state, const AttnParams& p) {
    TcState* st = static_cast<TcState*>(*state);
    if (!st) {
        st = new TcState();
        st->n_cached = st->next = 0;
        st->encode = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", reinterpret_cast<void**>(&st->encode), cudaEnableDefault, &qres);
        if (e != cudaSuccess || !st->encode) { delete st; return e != cudaSuccess ? e : cudaErrorNotSupported; }
        st->d = p.d; st->hkv = p.Hkv;
        if (p.d == 64) e = cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes);
        else e = cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes);
        if (e != cudaSuccess) { delete st; return e; }
        *state = st;
    }
    for (int i = 0; i < st->n_cached; ++i)
        if (st->cache[i].ptr == p.kv && st->cache[i].num_pages == p.num_pages) { st->current = &st->cache[i].map; return cudaSuccess; }
    TmapEntry& e = st->cache[st->next];
    cuuint64_t dims[2] = {(cuuint64_t)p.d, (cuuint64_t)p.num_pages * 2 * p.Hkv * 16};
    cuuint64_t strides[1] = {(cuuint64_t)p.d * 2};
    cuuint32_t box[2] = {64, 16};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = st->encode(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(p.kv), dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    e.ptr = p.kv;
    e.num_pages = p.num_pages;
    st->current = &e.map;
    st->next = (st->next + 1) % 64;
    if (st->n_cached < 64) ++st->n_cached;
    return cudaSuccess;
}

void launch_attn_tc(void* state, const AttnParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    const TcState* st = static_cast<const TcState*>(state);
    if (p.d == 64) attn_tc_kernel<64><<<p.n_ctas, kThreads, Cfg<64>::kSmemBytes, s>>>(*st->current, p);
    else attn_tc_kernel<128><<<p.n_ctas, kThreads, Cfg<128>::kSmemBytes, s>>>(*st->current, p);
}

void attn_tc_free(void* state) { delete static_cast<TcState*>(state); }

#ifdef FD_TRACE
// dst: [roles][per_role] packed events; counts: [roles].  Resets the counters.
extern "C" int fd_debug_read_trace(unsigned long long* dst, unsigned int* counts) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(counts, g_trace_n, sizeof(unsigned int) * kTraceRoles);
    cudaMemcpyFromSymbol(dst, g_trace, sizeof(unsigned long long) * kTraceRoles * kTracePerRole);
    unsigned int zero[kTraceRoles] = {0};
    cudaMemcpyToSymbol(g_trace_n, zero, sizeof(zero));
    return kTracePerRole;
}
#endif

}  // namespace fd
