// Internal declarations shared by the kernels of libflexdraft (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flexdraft.h"

namespace fd {

constexpr int kTileTokens = 128;   // KV tokens per work tile (8 pages of 16)
constexpr int kMaxRows = 128;      // query rows sharing one kv-head: G * Lq <= 128
constexpr int kAcceptChunk = 4096; // logits per CTA of the vocab sweep (smaller chunks measured faster: shorter CTA tails)

// Written by the plan kernel, read by the attention and merge kernels.
struct PlanHeader {
    int total_tiles;   // Hkv * sum_b tiles_b
    int fatal;         // lengths inconsistent: nothing is computed, out is zeroed
    int pad[2];
};

// Device-side view of the plan arrays (all live in the context's scratch memory).
struct Plan {
    PlanHeader* hdr;
    int* cu_q;      // [B+1] first query row of each sequence
    int* cu_tiles;  // [B+1] exclusive scan of tiles_b (per kv-head)
    int* seq_ok;    // [B]   0 = a page id of the sequence was outside the pool: its rows are zeroed
    int* seg_count; // [B * Hkv] partial pieces of a segment that have been written (fused merge)
    int* cta_first; // [n_ctas] sequence that owns the first tile of each attention CTA's range
};

// Partial result of one piece of a (sequence, kv-head) segment, log2 domain:
//   m[r] = max_j s2[r][j],  l[r] = sum_j exp2(s2[r][j] - m[r]),  O[r][c] = sum_j exp2(s2 - m) V[j][c]
// with s2 = scale * log2(e) * <q, k>.  Stored column-major (o[c * kMaxRows + r]) so that a
// thread-per-row kernel reads and writes it coalesced.
struct PartialView {
    float* o;  // [slots][d][kMaxRows]
    float* m;  // [slots][kMaxRows]
    float* l;  // [slots][kMaxRows]
};

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
    int n_ctas;       // CTAs of the attention grid (stream-K ranges are cut for this many)
    int* status;
};

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

// First tile of CTA c when `total` tiles are cut into `n` contiguous ranges.
__host__ __device__ inline int range_begin(int c, int total, int n) {
    return (int)(((long long)c * total) / n);
}
// The CTA whose range holds tile t.
__host__ __device__ inline int range_owner(int t, int total, int n) {
    return (int)((((long long)(t + 1)) * n + total - 1) / total) - 1;
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

// Number of partial pieces segment [t0, t1) was cut into by the CTA ranges (0 or 1 = not split).
__device__ inline int segment_pieces(int t0, int t1, int total, int n_ctas) {
    const int c_first = range_owner(t0, total, n_ctas), c_last = range_owner(t1 - 1, total, n_ctas);
    if (c_first == c_last) return 1;
    int n = 0;
    for (int c = c_first; c <= c_last; ++c) {
        const int sc = range_begin(c, total, n_ctas), ec = range_begin(c + 1, total, n_ctas);
        n += max(sc, t0) < min(ec, t1);
    }
    return n;
}

// Combine the partial pieces of segment (b, kvh) for query row r, columns [cg * CW, (cg + 1) * CW),
// in CTA-range order (fixed, so the result does not depend on timing), and write the bf16 output.
// The caller guarantees that every piece has been written and is visible.
template <int D, int CW>
__device__ inline void merge_row(const AttnParams& p, int total, int b, int kvh, int r, int cg) {
    const int row0 = p.plan.cu_q[b];
    __nv_bfloat16* dst = p.out + ((long long)(row0 + r / p.G) * p.Hq + kvh * p.G + r % p.G) * D + cg * CW;
    float acc[CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) acc[c] = 0.f;
    if (!__ldcg(p.plan.seq_ok + b)) {  // a page id of this sequence was bad: defined output, zeros
        store_cols_bf16<CW>(dst, acc, 0.f);
        return;
    }
    const int ntiles = p.plan.cu_tiles[b + 1] - p.plan.cu_tiles[b];
    const int t0 = p.Hkv * p.plan.cu_tiles[b] + kvh * ntiles, t1 = t0 + ntiles;
    const int c_first = range_owner(t0, total, p.n_ctas), c_last = range_owner(t1 - 1, total, p.n_ctas);
    float m = -INFINITY;
    for (int c = c_first; c <= c_last; ++c) {
        const int sc = range_begin(c, total, p.n_ctas), ec = range_begin(c + 1, total, p.n_ctas);
        if (max(sc, t0) >= min(ec, t1)) continue;
        const int slot = 2 * c + (sc >= t0 ? 0 : 1);
        m = fmaxf(m, __ldcg(p.part.m + slot * kMaxRows + r));
    }
    float l = 0.f;
    for (int c = c_first; c <= c_last; ++c) {
        const int sc = range_begin(c, total, p.n_ctas), ec = range_begin(c + 1, total, p.n_ctas);
        if (max(sc, t0) >= min(ec, t1)) continue;
        const int slot = 2 * c + (sc >= t0 ? 0 : 1);
        const float mp = __ldcg(p.part.m + slot * kMaxRows + r);
        if (mp == -INFINITY) continue;  // this piece saw no visible key for the row
        const float w = exp2f(mp - m);
        l += w * __ldcg(p.part.l + slot * kMaxRows + r);
        const float* o = p.part.o + ((long long)slot * D + cg * CW) * kMaxRows + r;
#pragma unroll
        for (int col = 0; col < CW; ++col) acc[col] += w * __ldcg(o + col * kMaxRows);
    }
    store_cols_bf16<CW>(dst, acc, 1.f / l);
}

// Launchers (defined next to their kernels).
void launch_plan(const AttnParams& p, cudaStream_t s);
cudaError_t attn_simt_prepare(int d);
void launch_attn_simt(const AttnParams& p, cudaStream_t s);
bool attn_tc_supported(int d, int G, int max_q_len);
cudaError_t attn_tc_prepare(void** state, const AttnParams& p);  // tensor map for this kv pool
void launch_attn_tc(void* state, const AttnParams& p, cudaStream_t s);
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
__device__ inline void fold(float& bv, unsigned& bi, float v, unsigned i) {
    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

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
};
void launch_accept(const AcceptParams& p, cudaStream_t s);

struct AppendParams {
    int batch, total_rows, num_pages, Hkv, d, max_pages;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* kv;
    const int32_t* page_table;
    const int32_t* prefix_lens;
    const int32_t* q_lens;
    int* status;
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
