// Draft-side tail of the step: calibrated argmax, confidence and the Eq. 5 verify length.
//
// One sweep over the [Rm, V] draft logits (+ bias).  A CTA owns one 4096-logit chunk of one row: it forms
// x = l + bias in fp32, reduces (max, argmax) to a 64-bit key and sum exp(x - chunk max), both in a fixed
// order, and stores them as the chunk's partial.  The CTA that delivers the last chunk of a row (a per-row
// counter, no spinning) combines the row's partials in a fixed order and writes token and confidence; the CTA
// that finishes last of all walks the cumulative confidence of every next-draft block against the threshold.
#include "fd_internal.cuh"

namespace fd {

constexpr int kDsVec = kAcceptChunk / (4 * 256);

// exp(x) for x <= 0 through one MUFU instruction (relative error about 2^-22: far inside the 1e-4 the
// confidences are compared at; the sweep is HBM-bound only if the per-element work stays this small)
constexpr float kLog2e = 1.4426950408889634f;
__device__ __forceinline__ float exp2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float exp_neg(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x * 1.4426950408889634f));
    return y;
}

// A chunk's partial from the 4 * kDsVec values each thread holds (thread t: elements 4 * (t + 256 * k) + q of the
// chunk [c0, c0 + n), -inf past the end): (max, argmax) as a key and sum exp(x - max), folded in a fixed order; thread
// 0 stores them.  `wkey`, `wsum`: 8 entries of shared memory each.  Holds one barrier.
__device__ __forceinline__ void ds_chunk_partial(const DraftSelectParams& p, const float (&x)[4 * kDsVec], int row, int chunk,
                                                 int chunks_per_row, int c0, int n, unsigned long long* wkey, float* wsum) {
    const int tid = threadIdx.x;
    // a thread meets its elements in index order, so "greater wins" keeps the lowest index of equal values;
    // padding (-inf) never wins, and a thread whose real elements are all -inf falls back to its first one
    float bv = -INFINITY;
    unsigned bi = 0xffffffffu;
#pragma unroll
    for (int k = 0; k < kDsVec; ++k)
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (x[4 * k + q] > bv) { bv = x[4 * k + q]; bi = (unsigned)(c0 + 4 * (tid + k * 256) + q); }
    if (bi == 0xffffffffu && 4 * tid < n) bi = (unsigned)(c0 + 4 * tid);
    unsigned long long key = (bi == 0xffffffffu) ? 0ull : make_key(bv, bi);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
    }
    // every warp: its maximum (as a key) and the sum of exp(x - that maximum); thread 0 folds the eight
    // pairs in warp order -- one barrier for the whole chunk
    // a warp wholly past the end of the row has key 0 and adds nothing; neither does one whose logits are all -inf
    // (a masked-out stretch of the vocabulary): its maximum must not enter a difference, -inf - -inf is NaN
    float mw = key ? key_value(key) : 0.f;
    if (mw == -INFINITY) mw = 0.f;
    float s = 0.f;
    const float nmw = -mw * kLog2e;
#pragma unroll
    for (int k = 0; k < kDsVec; ++k)
#pragma unroll
        for (int q = 0; q < 4; ++q)
            s += exp2_approx(fmaf(x[4 * k + q], kLog2e, nmw));  // one FMA per element; padding is -inf and adds 0
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((tid & 31) == 0) { wkey[tid >> 5] = key; wsum[tid >> 5] = s; }
    __syncthreads();
    if (tid == 0) {
        key = wkey[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) key = wkey[w] > key ? wkey[w] : key;
        const float m = key_value(key);  // chunk maximum (a chunk is never empty)
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w)
            if (wkey[w] && key_value(wkey[w]) > -INFINITY) t += wsum[w] * exp_neg(key_value(wkey[w]) - m);
        p.part_key[(long long)row * chunks_per_row + chunk] = key;
        p.part_sum[(long long)row * chunks_per_row + chunk] = t;
    }
}

// Warp 0 of the CTA that delivered the last chunk of `row` finishes the row.
__device__ __forceinline__ void ds_finish_row(const DraftSelectParams& p, int row, int chunks_per_row) {
    const int tid = threadIdx.x;
    if (tid < 32) {
        // the CTA that delivers the last chunk of a row finishes the row: lanes over chunks, maximum by an
        // exact reduction, sum of the rescaled chunk sums by a fixed shuffle tree (deterministic)
        __threadfence();
        const unsigned long long* pk = p.part_key + (long long)row * chunks_per_row;
        const float* ps = p.part_sum + (long long)row * chunks_per_row;
        unsigned long long best = 0ull;
        for (int c = tid; c < chunks_per_row; c += 32) { const unsigned long long k2 = __ldcg(pk + c); best = k2 > best ? k2 : best; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        const float mm = key_value(best);
        float tot = 0.f;
        for (int c = tid; c < chunks_per_row; c += 32) tot += __ldcg(ps + c) * exp_neg(key_value(__ldcg(pk + c)) - mm);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        if (tid == 0) {
            p.tokens[row] = key_index(best);
            p.probs[row] = 1.f / tot;
            p.row_ticket[row] = 0u;
        }
    }
}

// The CTA that finished last of all.  `m0`: batch + 1 ints of shared memory.
__device__ __forceinline__ void ds_final(const DraftSelectParams& p, int* m0) {
    const int tid = threadIdx.x;
    // ---- one CTA: rows -> (token, confidence), then blocks -> verify length
    __shared__ int carry, wcnt[8], s_bad;
    if (tid == 0) { carry = 0; m0[0] = 0; s_bad = 0; }
    __syncthreads();
    for (int base = 0; base < p.batch; base += blockDim.x) {
        const int b = base + tid;
        int v = 0;
        if (b < p.batch) {
            v = p.n_mask[b];
            const int nb = p.n_blocks ? p.n_blocks[b] : 1;
            if (v < 0 || nb < 0 || (nb > 1 && v % nb != 0) || max(nb, 1) > p.max_blocks) { atomicOr(&s_bad, 1); v = 0; }
        }
        int inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, inc, o);
            if ((tid & 31) >= o) inc += u;
        }
        if ((tid & 31) == 31) wcnt[tid >> 5] = inc;
        __syncthreads();
        int off = carry;
        for (int w = 0; w < (tid >> 5); ++w) off += wcnt[w];
        if (b < p.batch) m0[b + 1] = (int)min((long long)off + inc, (long long)0x7fffffff);
        __syncthreads();
        if (tid == blockDim.x - 1) carry = (int)min((long long)off + inc, (long long)0x7fffffff);
        __syncthreads();
    }
    if (tid == 0 && (s_bad || carry != p.total_rows)) { s_bad = 1; atomicOr(p.status, FD_DEV_BAD_LENGTHS); }
    __syncthreads();
    if (s_bad)
        for (int r = tid; r < p.total_rows; r += blockDim.x) { p.tokens[r] = -1; p.probs[r] = 0.f; }
    __syncthreads();
    for (int e = tid; e < p.batch * p.max_blocks; e += blockDim.x) {
        const int b = e / p.max_blocks, g = e % p.max_blocks;
        int keep = 0;
        if (!s_bad) {
            const int M = m0[b + 1] - m0[b], nb = max(p.n_blocks ? p.n_blocks[b] : 1, 1);
            if (M > 0 && g < nb) {
                const int kb = M / nb;
                const float* pr = p.probs + m0[b] + g * kb;  // written by other CTAs: read through L2
                float c = 1.f;
                bool open = true;
                for (int u0 = 0; u0 < kb && open; u0 += 8) {  // eight confidences per round trip, then the product in order
                    float v[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) v[k] = u0 + k < kb ? __ldcg(pr + u0 + k) : 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        c *= v[k];
                        if (open && u0 + k < kb && c >= p.threshold) ++keep; else open = false;
                    }
                }
            }
        }
        p.keep_len[e] = keep;
    }
    if (tid == 0) *p.ticket = 0u;
}

__global__ void __launch_bounds__(256, 8) draft_select_kernel(DraftSelectParams p, int chunks_per_row) {
    const int row = blockIdx.x / chunks_per_row, chunk = blockIdx.x % chunks_per_row;
    const long long rbase = (long long)row * p.vocab;
    const int c0 = chunk * kAcceptChunk, c1 = min(p.vocab, c0 + kAcceptChunk);
    const int tid = threadIdx.x, n = c1 - c0;
    const float* lg = p.logits + rbase + c0;
    const float* bs = p.bias ? p.bias + rbase + c0 : nullptr;
    const bool vec = (((reinterpret_cast<uintptr_t>(lg) | (bs ? reinterpret_cast<uintptr_t>(bs) : 0)) & 15) == 0);

    float x[4 * kDsVec];
#pragma unroll
    for (int k = 0; k < kDsVec; ++k) {
        const int e = 4 * (tid + k * 256);
        if (vec && e + 3 < n) {
            float4 a = __ldcs(reinterpret_cast<const float4*>(lg + e));
            if (bs) { const float4 b = __ldcs(reinterpret_cast<const float4*>(bs + e)); a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
            x[4 * k] = a.x; x[4 * k + 1] = a.y; x[4 * k + 2] = a.z; x[4 * k + 3] = a.w;
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) x[4 * k + q] = (e + q < n) ? (bs ? lg[e + q] + bs[e + q] : lg[e + q]) : -INFINITY;
        }
    }
    __shared__ unsigned long long wkey[8];
    __shared__ float wsum[8];
    __shared__ bool row_last, last;
    ds_chunk_partial(p, x, row, chunk, chunks_per_row, c0, n, wkey, wsum);
    if (tid == 0) {
        __threadfence();
        row_last = atomicAdd(p.row_ticket + row, 1u) == (unsigned)chunks_per_row - 1;
    }
    __syncthreads();
    if (!row_last) return;  // only the CTA that completes a row goes on: one fence + count per chunk, not two
    ds_finish_row(p, row, chunks_per_row);
    __syncthreads();
    if (tid == 0) {  // rows completed so far: whoever completes the last row finishes the call
        __threadfence();
        last = atomicAdd(p.ticket, 1u) == (unsigned)p.total_rows - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    // (behind an attention call the sweep has not waited for it; this one CTA does, before the call's last writes)
    if (p.chained) asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ int m0[];  // [B+1] first mask row of each sequence
    ds_final(p, m0);
}

// No mask rows at all: outputs are still defined.
__global__ void draft_select_empty_kernel(DraftSelectParams p) {
    bool bad = false;
    for (int b = 0; b < p.batch; ++b) bad |= p.n_mask[b] != 0;
    if (threadIdx.x == 0 && bad) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
    for (int e = threadIdx.x; e < p.batch * p.max_blocks; e += blockDim.x) p.keep_len[e] = 0;
}

void launch_draft_select(const DraftSelectParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    if (p.total_rows == 0) { draft_select_empty_kernel<<<1, 256, 0, s>>>(p); return; }
    const int chunks = (p.vocab + kAcceptChunk - 1) / kAcceptChunk;
    if (!p.chained) {
        draft_select_kernel<<<p.total_rows * chunks, 256, (p.batch + 1) * sizeof(int), s>>>(p, chunks);
        return;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.total_rows * chunks);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = (p.batch + 1) * sizeof(int);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, draft_select_kernel, p, chunks);
}

}  // namespace fd
