// Internal declarations shared by the kernels of libflexdraft (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flexdraft.h"

namespace fd {

constexpr int kTileTokens = 128;   // KV tokens per work tile (8 pages of 16)
constexpr int kMaxRows = 128;      // query rows sharing one kv-head: G * Lq <= 128
constexpr int kAcceptChunk = 8192; // logits per CTA of the vocab sweep

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
    int* seq_ok;    // [B]   0 = skipped (bad page id), 1 = computed
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
    __nv_bfloat16* out;
    Plan plan;
    PartialView part;
    int n_ctas;       // CTAs of the attention grid (stream-K ranges are cut for this many)
    int* status;
};

// First tile of CTA c when `total` tiles are cut into `n` contiguous ranges.
__host__ __device__ inline int range_begin(int c, int total, int n) {
    return (int)(((long long)c * total) / n);
}
// The CTA whose range holds tile t.
__host__ __device__ inline int range_owner(int t, int total, int n) {
    return (int)((((long long)(t + 1)) * n + total - 1) / total) - 1;
}

// Launchers (defined next to their kernels).
void launch_plan(const AttnParams& p, cudaStream_t s);
void launch_attn_simt(const AttnParams& p, cudaStream_t s);
bool attn_tc_supported(int d, int G, int max_q_len);
cudaError_t attn_tc_prepare(void** state, const AttnParams& p);  // tensor map for this kv pool
void launch_attn_tc(void* state, const AttnParams& p, cudaStream_t s);
void attn_tc_free(void* state);
void launch_merge(const AttnParams& p, cudaStream_t s);

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
