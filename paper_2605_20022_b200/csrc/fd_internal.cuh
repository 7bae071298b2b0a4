// Internal declarations shared by the kernels of libflexdraft (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flexdraft.h"

namespace fd {

constexpr int kTileTokens = 128;   // KV tokens per work tile (8 pages of 16)
constexpr int kMaxRows = 128;      // query rows of one MMA tile: a row block has kMaxRows / G block rows
constexpr int kClusterMaxSegments = 18; // most (sequence, kv-head) segments for which the kernel runs one cluster per segment
constexpr int kSelfPlanMaxRb = 24; // most row blocks for which the tensor-core kernel plans for itself (no plan launch)
constexpr int kAcceptChunk = 4096; // logits per CTA of the vocab sweep (smaller chunks measured faster: shorter CTA tails)

// Written by the plan kernel, read by the attention and merge kernels.
struct PlanHeader {
    int total_tiles;   // Hkv * sum over row blocks of their tiles
    int fatal;         // lengths inconsistent: nothing is computed, out is zeroed
    int n_rb;          // row blocks of the call
    int pad;
};

// A row block: up to rb_rows consecutive block rows of one sequence -- as many as fit the 128-row MMA tile
// together with their G q-heads.  A sequence whose query block is longer is handled as several row blocks,
// each streaming the sequence's KV on its own.  Everything the attention kernels index "per sequence" (scans,
// segments, piece counters) is per row block.
struct RowBlock {
    int b, i0;         // sequence, first block row
    int n, Lq, M, nb;  // the sequence's prefix length, query block length, mask tokens, mask blocks
    int pad[2];
};

// Device-side view of the plan arrays (all live in the context's scratch memory).
struct Plan {
    PlanHeader* hdr;
    RowBlock* rb;   // [n_rb] row blocks, sequence-major
    int* cu_q;      // [n_rb+1] first query row of each row block
    int* cu_tiles;  // [n_rb+1] exclusive scan of the row blocks' tiles (per kv-head)
    int* cu_ne;     // [n_rb+1] exclusive scan of (tiles > 0)
    int* seq_bad;   // [B]   number (AttnParams::epoch) of the last call that met a page id outside the pool in the sequence:
                    //       equal to the running call's number = flagged, the sequence's rows are zeroed
    int* seg_count; // [n_rb * Hkv][2] per segment: merge tickets drawn, partial pieces delivered (zero between calls)
    int* cta_first; // [n_ctas] row block that owns the first tile of each attention CTA's range
    int* cta_start; // [n_ctas + 1] first tile of each attention CTA's range (non-decreasing; [n_ctas] = total)
};

// Partial result of one piece of a (sequence, kv-head) segment, log2 domain:
//   m[r] = max_j s2[r][j],  l[r] = sum_j exp2(s2[r][j] - m[r]),  O[r][c] = sum_j exp2(s2 - m) V[j][c]
// with s2 = scale * log2(e) * <q, k>.  O is stored in groups of four columns, rows interleaved
// (o[(c / 4) * kMaxRows + r][c % 4]), so that a thread-per-row kernel moves it with 16-byte
// accesses that are contiguous across the warp.
struct PartialView {
    float* o;  // [slots][d / 4][kMaxRows][4]
    float* m;  // [slots][kMaxRows]
    float* l;  // [slots][kMaxRows]
};

// Where row r of partial `slot` keeps columns [col, col + 4) (col a multiple of 4); the next four columns
// are kMaxRows float4 further on.
__device__ __forceinline__ float4* partial_o4(const PartialView& part, int d, int slot, int col, int r) {
    return reinterpret_cast<float4*>(part.o) + ((long long)slot * (d / 4) + (col >> 2)) * kMaxRows + r;
}

struct AttnParams {
    int batch, total_q_rows, num_pages;
    int Hq, Hkv, G, d, max_pages, max_q_len;
    float scale_log2e;
    const __nv_bfloat16* q;
    const __nv_bfloat16* kv;
    const int32_t* page_table;
    const int32_t* prefix_lens;
    const int32_t* q_lens;
    const int32_t* n_mask;
    const int32_t* n_blocks;  // [B] mask blocks per sequence, or nullptr (= one block each)
    __nv_bfloat16* out;
    Plan plan;
    PartialView part;
    int rb_rows;      // block rows per row block: kMaxRows / G
    int rb_per_seq;   // most row blocks a sequence can have: ceil(max_q_len / rb_rows)
    int max_rb;       // capacity of the row-block arrays
    int n_ctas;       // CTAs of the attention grid (stream-K ranges are cut for this many)
    int q_box_t;      // block rows per Q load box of the tensor-core kernel (see q_box_rows)
    int min_range_tiles;  // least tiles worth giving a CTA a range of its own
    int piece_cost;   // fixed cost of starting a segment in a range, in tiles (balances ranges with many short segments)
    int epoch;        // number of this attention call on its context, never 0 (see Plan::seq_bad)
    int cluster;      // CTAs per cluster when every segment is split over one cluster, else 0
    int early;        // 1: the launch before this one on the stream is an attention or append call served by the same pinned
                      //    plan, which writes neither the plan nor the lengths nor the page table: they may be read
                      //    before that launch has completed (everything else waits for it)
                      // 2: nor does any call of that chain write q or the cache of this one: they may be read early too,
                      //    and the first piece worked through; the call waits before its first write to global memory
                      // 3: as 2, but the launch before this one is the KV append of this cache: tiles of the prefix are
                      //    read early, a tile that reaches into the query block after the wait
    int* status;
};

// A sequence in which this call met a page id outside the pool: its rows are written as zeros.  The flag is the
// call's own number, so nothing has to be cleared between calls.
__device__ __forceinline__ void flag_sequence(const AttnParams& p, int b) {
    p.plan.seq_bad[b] = p.epoch;
    atomicOr(p.status, FD_DEV_BAD_PAGE);
}
__device__ __forceinline__ bool sequence_flagged(const AttnParams& p, int b) { return __ldcg(p.plan.seq_bad + b) == p.epoch; }

// Hybrid mask of one query row, never materialised: key position j is visible iff
//     j < limit  ||  (blk_lo <= j && j < blk_hi).
// Candidate row i: causal (limit = n + i + 1, no block).  Mask row of block g (of nb blocks of M / nb
// tokens): the branch prepared under the hypothesis "r = C - nb + g drafts accepted" sees the prefix and
// the candidates 0..r (limit = n + r + 1) and its own block in both directions; with nb = 1 that is
// every key of the sequence.  Rows that do not exist see nothing.
struct RowMask {
    int limit, blk_lo, blk_hi;
};
__host__ __device__ inline RowMask row_mask(int i, int n, int Lq, int M, int nb, bool exists) {
    RowMask rm = {0, 0, 0};
    if (!exists) return rm;
    const int C = Lq - M;
    if (i < C) { rm.limit = n + i + 1; return rm; }
    if (nb < 1) nb = 1;
    const int kb = M / nb, g = (i - C) / kb;
    rm.limit = n + (C - nb + g) + 1;
    rm.blk_lo = n + C + g * kb;
    rm.blk_hi = rm.blk_lo + kb;
    return rm;
}

// Block rows one Q load brings in: the largest power of two <= 8 that divides the most block rows a
// segment can have (kMaxRows / G), so that rounding a block length up to whole boxes never passes the tile.
__host__ __device__ inline int q_box_rows(int G) {
    int bt = 8;
    while ((kMaxRows / G) % bt) bt >>= 1;
    return bt;
}

// Range cutting (host and device).  Cost position x of a tile: Hkv * (tiles + k * segments started) before
// it, with a segment's k start-up units ahead of its tiles.  A call worth W units is spread over
//     n_use = clamp(W / (k + min_range_tiles), 1, n_ranges)
// ranges; range c starts at the tile that holds x = c * W / n_use (a position inside the start-up units
// snaps to the segment's first tile).  ct_at(b) / ne_at(b): exclusive scans over the sequences of tiles
// per kv-head and of "has tiles".  Returns the first tile of range c; *first_seq = the sequence it lies in.
__host__ __device__ inline int ranges_in_use(long long W, long long k, int min_range_tiles, int n_ranges) {
    const long long per = k + (min_range_tiles > 1 ? min_range_tiles : 1);
    long long n = ((unsigned long long)W >> 32) == 0 ? (long long)((unsigned)W / (unsigned)per) : W / per;
    if (n > n_ranges) n = n_ranges;
    return (int)(n < 1 ? 1 : n);
}
template <class CtAt, class NeAt>
__host__ __device__ inline int range_cut(int c, int n_use, long long W, int B, int Hkv, long long k, CtAt ct_at, NeAt ne_at,
                                         int* first_seq) {
    // (64-bit division is a long dependent instruction sequence on the device: the 32-bit form serves every call
    // whose cost total fits, with the same result)
    const unsigned long long cw = (unsigned long long)c * (unsigned long long)W;
    const long long x = (cw >> 32) == 0 ? (long long)((unsigned)cw / (unsigned)n_use) : (long long)(cw / (unsigned long long)n_use);
    int lo = 0, hi = B;  // last b whose span starts at or before x (of equal starts the last: the non-empty one)
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        const long long w_mid = (long long)Hkv * ((long long)ct_at(mid) + k * (long long)ne_at(mid));
        if (w_mid <= x) lo = mid; else hi = mid;
    }
    const long long ct = ct_at(lo), nt = (long long)ct_at(lo + 1) - ct;
    const long long rem = x - (long long)Hkv * (ct + k * (long long)ne_at(lo));
    long long kvh, r;
    if (((unsigned long long)rem >> 32) == 0 && ((unsigned long long)(nt + k) >> 32) == 0) {
        kvh = (unsigned)rem / (unsigned)(nt + k);
        r = (unsigned)rem - (unsigned)kvh * (unsigned)(nt + k);
    } else {
        kvh = rem / (nt + k);
        r = rem % (nt + k);
    }
    *first_seq = lo;
    return (int)(Hkv * ct + kvh * nt + (r > k ? r - k : 0));
}

// View of the range starts cta_start[c]: a window around the reading CTA may be cached in shared memory; an entry
// outside the window comes from the plan kernel's array in global memory, or -- in a call that plans for itself
// and has no such array -- is cut again from the scans (ct, ne: tiles and non-empty row blocks, exclusive).
constexpr int kCsWindow = 32;
struct CtaStarts {
    const int* g;   // [n_ctas + 1] in global memory, or nullptr
    const int* s;   // entries [base, base + kCsWindow) in shared memory, or nullptr
    int base;
    const int* ct;  // self-planned call: [n_rb + 1] scans, and what range_cut needs beside them
    const int* ne;
    int n_rb, Hkv, n_use, k, total;
    long long W;
    __device__ __forceinline__ int cut(int c) const {
        if (c >= n_use) return total;
        int first;
        const int* ct_ = ct;
        const int* ne_ = ne;
        return range_cut(c, n_use, W, n_rb, Hkv, (long long)k, [ct_](int b) { return ct_[b]; }, [ne_](int b) { return ne_[b]; }, &first);
    }
    __device__ __forceinline__ int at(int c) const {
        const unsigned i = (unsigned)(c - base);
        if (s && i < (unsigned)kCsWindow) return s[i];
        return g ? g[c] : cut(c);
    }
};

// The CTA whose range [cta_start[c], cta_start[c + 1]) holds tile t (ranges may be empty: of several CTAs
// that start at the same tile the last one is the one that owns it).
__device__ inline int range_owner(const int* cta_start, int n_ctas, int t) {
    int lo = 0, hi = n_ctas;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cta_start[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// First and last CTA whose range meets segment [t0, t1), found by walking outwards from `c`, a CTA that is
// known to meet it (a segment rarely spans more than a few ranges).
__device__ inline void segment_ctas(const CtaStarts& cs, int n_ctas, int c, int t0, int t1, int& c_first, int& c_last) {
    c_first = c_last = c;
    while (c_first > 0 && cs.at(c_first) > t0) --c_first;
    while (c_last + 1 < n_ctas && cs.at(c_last + 1) < t1) ++c_last;
}

// Number of partial pieces the CTAs c_first..c_last hold of segment [t0, t1) (1 = not split).
__device__ inline int segment_pieces(const CtaStarts& cs, int c_first, int c_last, int t0, int t1) {
    int n = 0;
    for (int c = c_first; c <= c_last; ++c) n += max(cs.at(c), t0) < min(cs.at(c + 1), t1);
    return n;
}

// Write one row segment of `n` columns as bf16 (n a multiple of 8), scaled by inv.
template <int N>
__device__ inline void store_cols_bf16(__nv_bfloat16* dst, const float* o, float inv) {
#pragma unroll
    for (int c = 0; c < N; c += 8) {
        __align__(16) __nv_bfloat162 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = __floats2bfloat162_rn(o[c + 2 * k] * inv, o[c + 2 * k + 1] * inv);
        *reinterpret_cast<uint4*>(dst + c) = *reinterpret_cast<const uint4*>(v);
    }
}

// Combine the partial pieces of segment (b, kvh) = tiles [t0, t1), held by CTAs c_first..c_last, for query
// row r (output row row0 + r / G), columns [cg * CW, (cg + 1) * CW), in CTA order (fixed, so the result does
// not depend on timing), and write the bf16 output.  The caller guarantees that every piece has been
// written and is visible.  A piece that saw no visible key for the row holds m = -inf, l = 0, O = 0.
// `own` (or nullptr): the O values of CTA own_cta's piece for exactly this row and these columns, still in
// the caller's registers -- the same numbers it stored, so using them instead of loading changes nothing.
template <int D, int CW>
__device__ inline void merge_row(const AttnParams& p, const CtaStarts& cs, int c_first, int c_last, int b, int kvh, int row0,
                                 int t0, int t1, int r, int cg, const float* own = nullptr, int own_cta = -1) {
    __nv_bfloat16* dst = p.out + ((long long)(row0 + r / p.G) * p.Hq + kvh * p.G + r % p.G) * D + cg * CW;
    float acc[CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) acc[c] = 0.f;
    if (sequence_flagged(p, b)) {  // a page id of this sequence was bad: defined output, zeros
        store_cols_bf16<CW>(dst, acc, 0.f);
        return;
    }
    float m = -INFINITY;
    for (int c = c_first; c <= c_last; ++c) {
        const int sc = cs.at(c), ec = cs.at(c + 1);
        if (max(sc, t0) >= min(ec, t1)) continue;
        const int slot = 2 * c + (sc >= t0 ? 0 : 1);
        m = fmaxf(m, __ldcg(p.part.m + slot * kMaxRows + r));
    }
    float l = 0.f;
    for (int c = c_first; c <= c_last; ++c) {
        const int sc = cs.at(c), ec = cs.at(c + 1);
        if (max(sc, t0) >= min(ec, t1)) continue;
        const int slot = 2 * c + (sc >= t0 ? 0 : 1);
        const float mp = __ldcg(p.part.m + slot * kMaxRows + r);
        const float lp = __ldcg(p.part.l + slot * kMaxRows + r);
        const float4* o = partial_o4(p.part, D, slot, cg * CW, r);
        const float w = (mp == -INFINITY) ? 0.f : exp2f(mp - m);
        l += w * lp;
        if (own && c == own_cta) {
#pragma unroll
            for (int k = 0; k < CW; ++k) acc[k] += w * own[k];
            continue;
        }
        float4 v[CW / 4];  // independent 16-byte loads, all in flight together
#pragma unroll
        for (int k = 0; k < CW / 4; ++k) v[k] = __ldcg(o + k * kMaxRows);
#pragma unroll
        for (int k = 0; k < CW / 4; ++k) {
            acc[4 * k] += w * v[k].x;
            acc[4 * k + 1] += w * v[k].y;
            acc[4 * k + 2] += w * v[k].z;
            acc[4 * k + 3] += w * v[k].w;
        }
    }
    store_cols_bf16<CW>(dst, acc, 1.f / l);
}

// How a tensor-core attention call finds its work: from the plan kernel's arrays; from scans each CTA makes
// itself (few row blocks); or one cluster per segment, merged through distributed shared memory.
enum { kTcPlanned = 0, kTcSelfPlanned = 1, kTcCluster = 2 };

// Launchers (defined next to their kernels).
void launch_plan(const AttnParams& p, cudaStream_t s);
cudaError_t attn_simt_prepare(int d);
void launch_attn_simt(const AttnParams& p, cudaStream_t s);
bool attn_tc_supported(int d, int G, int max_q_len);
cudaError_t attn_tc_prepare(void** state, const AttnParams& p);  // tensor map for this kv pool
void launch_attn_tc(void* state, const AttnParams& p, int mode, cudaStream_t s);  // mode: kTcPlanned, kTcSelfPlanned, kTcCluster
int attn_tc_cluster_size(const void* state, int n_segments, int n_sms);    // CTAs per cluster for a call of n_segments, or 0
void attn_tc_free(void* state);
void launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, cudaStream_t s);
void launch_merge(const AttnParams& p, cudaStream_t s);

// (value, index) of a running argmax as one 64-bit key: order-preserving image of the float in the high
// word, inverted index in the low word, so an unsigned max picks the larger value and, on equal values,
// the lower index.  A key of 0 means "nothing seen".
__device__ inline unsigned long long make_key(float v, unsigned idx) {
    v += 0.0f;  // -0.0 -> +0.0: they compare equal, so the lower index must decide
    unsigned u = __float_as_uint(v);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (unsigned long long)(0xffffffffu - idx);
}
__device__ inline float key_value(unsigned long long key) {
    const unsigned u = (unsigned)(key >> 32);
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}
__device__ inline int key_index(unsigned long long key) { return (int)(0xffffffffu - (unsigned)(key & 0xffffffffull)); }

struct DraftSelectParams {
    int batch, total_rows, vocab, max_blocks;
    const float* logits;
    const float* bias;        // may be nullptr
    const int32_t* n_mask;
    const int32_t* n_blocks;  // may be nullptr
    float threshold;
    int32_t* tokens;
    float* probs;
    int32_t* keep_len;        // [B, max_blocks]
    int chained;                   // 1: behind an attention call, as AcceptParams::chained (the sweep runs ahead)
    unsigned long long* part_key;  // [rows][chunks] per-chunk (max, argmax)
    float* part_sum;               // [rows][chunks] per-chunk sum of exp(x - chunk max)
    unsigned int* ticket;
    unsigned int* row_ticket;      // [rows] chunks of the row delivered so far (zero between calls)
    int* status;
};
void launch_draft_select(const DraftSelectParams& p, cudaStream_t s);

struct AcceptParams {
    int batch, total_rows, vocab;
    const float* logits;
    const int32_t* drafts;
    const int32_t* q_lens;
    const int32_t* n_mask;
    int32_t* accepted;
    int32_t* bonus;
    unsigned long long* keys;  // [max rows] running (value, index) maxima, zero between calls
    unsigned int* ticket;      // [1] CTAs finished, zero between calls
    int* status;
    int chained;               // 1: launched as a programmatic dependent of the attention call before it: the sweep -- logits
                               //    in, private scratch out -- runs while that call finishes; the CTA that finishes last
                               //    waits for it before the scan writes the results
};
void launch_accept(const AcceptParams& p, cudaStream_t s);

struct SampleParams {
    int batch, total_rows, vocab;
    float kt;                      // log2(e) / temperature
    const float* logits;
    const float* draft_logits;     // may be nullptr: all mass on the proposed token
    const int32_t* drafts;
    const int32_t* q_lens;
    const int32_t* n_mask;
    const float* u_accept;
    const float* u_bonus;
    int32_t* accepted;
    int32_t* bonus;
    float2* part;                  // [rows][chunks][2] chunk (max, sum) of the target and of the draft row
    float2* row_stat;              // [rows][2] row (max, Z)
    unsigned int* row_ticket;      // [rows], zero between calls
    unsigned int* ticket;          // [1], zero between calls
    int4* seq_info;                // [B] (row the bonus is drawn from, mode, rejected token, -)
    float* chunk_w;                // [B][chunks] weight sums
    unsigned int* seq_ticket;      // [B], zero between calls
    unsigned char* flags;          // [rows] accept test passed
    int* status;
    int chained;                   // 1: behind an attention call, as AcceptParams::chained (the statistics sweep runs ahead)
};
int launch_accept_sample(const SampleParams& p, cudaStream_t s);  // returns the number of kernels launched

struct AppendParams {
    int batch, total_rows, num_pages, Hkv, d, max_pages, max_q_len;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* kv;
    const int32_t* page_table;
    const int32_t* prefix_lens;
    const int32_t* q_lens;
    int* status;
    int chained;  // 1: launched as a programmatic dependent of an attention call of the same pinned chain, none of whose
                  //    writes it reads: the copies run while that call finishes, the kernel waits for it before it ends
};
void launch_kv_append(const AppendParams& p, cudaStream_t s);

struct SelectParams {
    int batch, max_kb;
    const int32_t* mask_tokens;
    const int32_t* q_lens;
    const int32_t* n_mask;
    const int32_t* n_blocks;  // may be nullptr
    const int32_t* accepted;
    int32_t* next_draft;
    int32_t* next_len;
    int* status;
};
void launch_select_branch(const SelectParams& p, cudaStream_t s);

struct CommitParams {
    int batch, max_pages, page_size;
    int32_t* page_table;
    int32_t* prefix_lens;
    const int32_t* q_lens;
    const int32_t* accepted;
    int32_t* freed;
    int32_t* n_freed;
    int* status;
};
void launch_commit(const CommitParams& p, cudaStream_t s);

}  // namespace fd
