// Greedy verification: vocab argmax of every candidate row fused with the accept scan.
//
// The [R, V] fp32 logits are swept once.  Each CTA reduces one 4096-logit chunk of one row
// to a 64-bit key (order-preserving image of the float in the high word, ~index in the low
// word, so an unsigned max picks the larger value and, on equal values, the lower index)
// and folds it into the row's running key with atomicMax -- an exact, order-independent
// reduction, so the result is deterministic.  The CTA that finishes last (a ticket counter,
// no spinning) runs the per-sequence accept scan and re-zeroes the keys for the next call.
#include "fd_internal.cuh"

namespace fd {

constexpr int kVecPerThread = kAcceptChunk / (4 * 256);  // float4 loads in flight per thread

// The accept scan: one CTA of 256 threads, after every row key is final.  `sm`: 2 * batch + 1 ints of shared memory.
__device__ __forceinline__ void accept_scan(const AcceptParams& p, int* sm) {
    const int tid = threadIdx.x;

    // ---- accept scan, one CTA, after every row key is final.  Everything is one parallel round of
    //      loads per step (serial walks over global memory would cost a DRAM/L2 latency per element):
    //      (1) block scan of the candidate-row counts, (2) one thread per candidate row compares its
    //      argmax with the next draft and lowers the sequence's first-mismatch index, (3) one thread
    //      per sequence reads the argmax at that index.
    int* cu_c = sm;
    int* first_bad = sm + p.batch + 1;
    __shared__ int s_bad, s_carry, s_wsum[8];
    if (tid == 0) { s_bad = 0; s_carry = 0; cu_c[0] = 0; }
    __syncthreads();
    for (int base = 0; base < p.batch; base += blockDim.x) {
        const int b = base + tid;
        int c = 0;
        if (b < p.batch) {
            const int M = p.n_mask[b];
            c = p.q_lens[b] - M;
            if (c < 0 || M < 0) { atomicOr(&s_bad, 1); c = 0; }
        }
        int inc = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, inc, o);
            if ((tid & 31) >= o) inc += u;
        }
        if ((tid & 31) == 31) s_wsum[tid >> 5] = inc;
        __syncthreads();
        int off = s_carry;
        for (int w = 0; w < (tid >> 5); ++w) off += s_wsum[w];
        if (b < p.batch) {
            const long long end = (long long)off + inc;
            cu_c[b + 1] = (int)min(end, (long long)0x7fffffff);
            first_bad[b] = max(c - 1, 0);                      // k_b: "every draft matched"
        }
        __syncthreads();
        if (tid == blockDim.x - 1) s_carry = min((long long)off + inc, (long long)0x7fffffff);
        __syncthreads();
    }
    if (tid == 0 && (s_bad || s_carry != p.total_rows)) { s_bad = 1; atomicOr(p.status, FD_DEV_BAD_LENGTHS); }
    __syncthreads();
    if (s_bad) {
        for (int b = tid; b < p.batch; b += blockDim.x) { p.accepted[b] = -1; p.bonus[b] = -1; }
    } else {
        for (int r = tid; r < p.total_rows; r += blockDim.x) {
            int lo = 0, hi = p.batch;                          // sequence of row r: last b with cu_c[b] <= r
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (cu_c[mid] <= r) lo = mid; else hi = mid;
            }
            const int j = r - cu_c[lo];
            if (r + 1 < cu_c[lo + 1]) {                        // row j has a draft after it
                const int am = (int)(0xffffffffu - (unsigned)(__ldcg(p.keys + r) & 0xffffffffull));
                if (am != p.drafts[r + 1]) atomicMin(&first_bad[lo], j);
            }
        }
        __syncthreads();
        for (int b = tid; b < p.batch; b += blockDim.x) {
            const int r0 = cu_c[b], C = cu_c[b + 1] - r0;
            if (C == 0) { p.accepted[b] = -1; p.bonus[b] = -1; continue; }
            const int a = first_bad[b];
            p.accepted[b] = a;
            p.bonus[b] = (int)(0xffffffffu - (unsigned)(__ldcg(p.keys + r0 + a) & 0xffffffffull));
        }
    }
    __syncthreads();
    for (int r = tid; r < p.total_rows; r += blockDim.x) p.keys[r] = 0ull;
    if (tid == 0) *p.ticket = 0u;
}

__global__ void __launch_bounds__(256) accept_kernel(AcceptParams p, int chunks_per_row) {
    const int row = blockIdx.x / chunks_per_row, chunk = blockIdx.x % chunks_per_row;
    const float* base = p.logits + (long long)row * p.vocab;
    const int c0 = chunk * kAcceptChunk, c1 = min(p.vocab, c0 + kAcceptChunk);
    const int tid = threadIdx.x;

    // A thread meets its elements in index order (head, body, tail), so "greater wins" keeps the lowest index of
    // equal values; a thread whose elements are all -inf falls back to the first one it owns.
    float bv = -INFINITY;
    unsigned bi = 0xffffffffu, first = 0xffffffffu;
    // scalar head up to the first 16-byte boundary, float4 body, scalar tail
    const int mis = (int)((reinterpret_cast<uintptr_t>(base + c0) >> 2) & 3);
    const int head = min(c1 - c0, (4 - mis) & 3);
    const int nvec = (c1 - c0 - head) >> 2;
    if (tid < head) { first = c0 + tid; const float v0 = base[c0 + tid]; if (v0 > bv) { bv = v0; bi = c0 + tid; } }
    const float4* vp = reinterpret_cast<const float4*>(base + c0 + head);
    float4 v[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int e = tid + k * 256;
        v[k] = (e < nvec) ? __ldcs(vp + e) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
    if (first == 0xffffffffu && tid < nvec) first = c0 + head + 4 * tid;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {  // padding is -inf and never wins
        const unsigned i0 = c0 + head + 4 * (tid + k * 256);
        if (v[k].x > bv) { bv = v[k].x; bi = i0; }
        if (v[k].y > bv) { bv = v[k].y; bi = i0 + 1; }
        if (v[k].z > bv) { bv = v[k].z; bi = i0 + 2; }
        if (v[k].w > bv) { bv = v[k].w; bi = i0 + 3; }
    }
    const int tail0 = c0 + head + 4 * nvec;
    if (tail0 + tid < c1) {
        if (first == 0xffffffffu) first = tail0 + tid;
        const float vt = base[tail0 + tid];
        if (vt > bv) { bv = vt; bi = tail0 + tid; }
    }
    if (bi == 0xffffffffu) bi = first;

    unsigned long long key = (bi == 0xffffffffu) ? 0ull : make_key(bv, bi);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
    }
    __shared__ unsigned long long wkey[8];
    __shared__ bool last;
    if ((tid & 31) == 0) wkey[tid >> 5] = key;
    __syncthreads();
    if (tid == 0) {
#pragma unroll
        for (int w = 1; w < 8; ++w) key = wkey[w] > key ? wkey[w] : key;
        atomicMax(p.keys + row, key);
        __threadfence();
        last = atomicAdd(p.ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    // (one CTA that waits is enough to keep this launch from completing before the one it was chained to)
    if (p.chained) asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ int sm[];            // cu_c [B+1], then first_mismatch [B]
    accept_scan(p, sm);
}

// R = 0: nothing to sweep, but the outputs are still defined (-1 everywhere).
__global__ void accept_empty_kernel(AcceptParams p) {
    bool bad = false;
    for (int b = 0; b < p.batch; ++b) bad |= (p.q_lens[b] - p.n_mask[b]) != 0;
    if (threadIdx.x == 0 && bad) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
    for (int b = threadIdx.x; b < p.batch; b += blockDim.x) { p.accepted[b] = -1; p.bonus[b] = -1; }
}

void launch_accept(const AcceptParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    if (p.total_rows == 0) { accept_empty_kernel<<<1, 256, 0, s>>>(p); return; }
    const int chunks = (p.vocab + kAcceptChunk - 1) / kAcceptChunk;
    if (!p.chained) {
        accept_kernel<<<p.total_rows * chunks, 256, (2 * p.batch + 1) * sizeof(int), s>>>(p, chunks);
        return;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.total_rows * chunks);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = (2 * p.batch + 1) * sizeof(int);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, accept_kernel, p, chunks);
}

}  // namespace fd
