// KV commit / rollback: length truncation and page release, one CTA.
#include <algorithm>

#include "fd_internal.cuh"

namespace fd {

// How many pages sequence b gives back, or -1 if its entry is inconsistent (left unchanged), 0 if it takes no part.
__device__ __forceinline__ int pages_released(const CommitParams& p, int b, int& a, int& n, int& Lq) {
    const int P = p.page_size;
    a = p.accepted[b]; Lq = p.q_lens[b]; n = p.prefix_lens[b];
    if (a < 0) return 0;
    if (a >= Lq || Lq < 0 || n < 0 || (long long)n + Lq > (long long)p.max_pages * P) return -1;
    return (n + Lq + P - 1) / P - (n + a + 1 + P - 1) / P;
}

__global__ void __launch_bounds__(256) commit_kernel(CommitParams p) {
    __shared__ int wsum[8], carry;
    const int tid = threadIdx.x, P = p.page_size;
    if (tid == 0) carry = 0;
    __syncthreads();
    // sequences in chunks of 256: block scan of the pages each gives back -> its place in the freed list
    for (int base = 0; base < p.batch; base += blockDim.x) {
        const int b = base + tid;
        int a = -1, n = 0, Lq = 0, cnt = 0;
        if (b < p.batch) {
            cnt = pages_released(p, b, a, n, Lq);
            if (cnt < 0) atomicOr(p.status, FD_DEV_BAD_ACCEPT);
        }
        const int mine = max(cnt, 0);
        int inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, inc, o);
            if ((tid & 31) >= o) inc += u;
        }
        if ((tid & 31) == 31) wsum[tid >> 5] = inc;
        __syncthreads();
        int off = carry;
        for (int w = 0; w < (tid >> 5); ++w) off += wsum[w];
        off += inc - mine;
        if (b < p.batch && a >= 0 && cnt >= 0) {
            const int new_len = n + a + 1;
            const int keep = (new_len + P - 1) / P;
            int32_t* row = p.page_table + (long long)b * p.max_pages;
            for (int k = 0; k < cnt; ++k) {
                p.freed[off + k] = row[keep + k];
                row[keep + k] = -1;
            }
            p.prefix_lens[b] = new_len;
        }
        __syncthreads();
        if (tid == blockDim.x - 1) carry = off + mine;
        __syncthreads();
    }
    if (tid == 0) *p.n_freed = carry;
}

void launch_commit(const CommitParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    commit_kernel<<<1, 256, 0, s>>>(p);
}

// KV append: K/V of the query block -> its pages ("append, then attend").  A CTA per (sequence, group of block rows);
// 16-byte copies, one page lookup per row.  (One CTA per sequence took 15 us for a 32-row block: 32 dependent rounds.)
__global__ void __launch_bounds__(256) kv_append_kernel(AppendParams p, int rows_per_cta) {
    // the attention call that follows on the stream may start its set-up now; it waits for this grid to complete
    // before it reads the cache
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ int s_red[8];
    __shared__ long long s_row0;
    const int b = blockIdx.x, i0 = blockIdx.y * rows_per_cta, tid = threadIdx.x;
    const int n = p.prefix_lens[b], Lq = p.q_lens[b];
    // (p.chained: the launch before this one may still be running -- it writes nothing this kernel reads; every CTA
    // waits for it before leaving, so that whoever waits for THIS launch has waited for that one too)
    if (i0 >= Lq) {  // uniform (an empty or negative length too)
        if (p.chained) asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    // first query row of this sequence = sum of the lengths before it (block-parallel; negative lengths count as 0)
    int part = 0;
    for (int s = tid; s < b; s += blockDim.x) part += max(p.q_lens[s], 0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if ((tid & 31) == 0) s_red[tid >> 5] = part;
    __syncthreads();
    if (tid == 0) {
        long long r = 0;
        for (int w = 0; w < 8; ++w) r += s_red[w];
        s_row0 = r;
    }
    __syncthreads();
    const long long row0 = s_row0;
    if (n < 0 || row0 + Lq > p.total_rows || (long long)n + Lq > (long long)p.max_pages * 16) {
        if (p.chained) asm volatile("griddepcontrol.wait;" ::: "memory");  // (before the write to the status word, too)
        if (tid == 0 && i0 == 0) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
        return;
    }
    const int vec_per_head = p.d / 8;                    // 16-byte pieces of one head's row
    const int per_row = p.Hkv * vec_per_head;
    const int i1 = min(Lq, i0 + rows_per_cta);
    bool bad_page = false;
    for (int i = i0; i < i1; ++i) {
        const int j = n + i;
        const int page = p.page_table[(long long)b * p.max_pages + (j >> 4)];
        if ((unsigned)page >= (unsigned)p.num_pages) {   // never form an address from a bad id
            bad_page = true;  // (reported at the end: the status word is shared with the launch before this one)
            continue;
        }
        for (int e = tid; e < 2 * per_row; e += blockDim.x) {
            const int which = e / per_row, rem = e % per_row;
            const int h = rem / vec_per_head, v = rem % vec_per_head;
            const __nv_bfloat16* src = (which ? p.v_new : p.k_new) + ((row0 + i) * p.Hkv + h) * p.d + v * 8;
            __nv_bfloat16* dst = p.kv + ((((long long)page * 2 + which) * p.Hkv + h) * 16 + (j & 15)) * p.d + v * 8;
            *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
        }
    }
    if (p.chained) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (bad_page && tid == 0) atomicOr(p.status, FD_DEV_BAD_PAGE);
}

void launch_kv_append(const AppendParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    // a handful of rows per CTA; long query blocks (up to 4096 rows) get more rows per CTA instead of more CTAs
    const int rows_per_cta = std::max(4, (p.max_q_len + 63) / 64);
    const int groups = (p.max_q_len + rows_per_cta - 1) / rows_per_cta;
    if (!p.chained) {
        kv_append_kernel<<<dim3(p.batch, groups), 256, 0, s>>>(p, rows_per_cta);
        return;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.batch, groups);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kv_append_kernel, p, rows_per_cta);
}

// Branch selection after verification (parallel drafting with one prepared branch per hypothesis):
// copy the tokens of the block prepared for r = accepted_len drafts accepted.  One CTA.
__global__ void __launch_bounds__(256) select_branch_kernel(SelectParams p) {
    extern __shared__ int m0[];  // [B+1] exclusive scan of n_mask
    __shared__ int carry, wsum[8];
    const int tid = threadIdx.x;
    if (tid == 0) { carry = 0; m0[0] = 0; }
    __syncthreads();
    for (int base = 0; base < p.batch; base += blockDim.x) {
        const int b = base + tid;
        int v = (b < p.batch) ? max(p.n_mask[b], 0) : 0, inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, inc, o);
            if ((tid & 31) >= o) inc += u;
        }
        if ((tid & 31) == 31) wsum[tid >> 5] = inc;
        __syncthreads();
        int off = carry;
        for (int w = 0; w < (tid >> 5); ++w) off += wsum[w];
        if (b < p.batch) m0[b + 1] = off + inc;
        __syncthreads();
        if (tid == blockDim.x - 1) carry = off + inc;
        __syncthreads();
    }
    for (int e = tid; e < p.batch * p.max_kb; e += blockDim.x) {
        const int b = e / p.max_kb, u = e % p.max_kb;
        const int M = p.n_mask[b], C = p.q_lens[b] - M, a = p.accepted[b];
        int nb = p.n_blocks ? p.n_blocks[b] : 1;
        if (nb < 1) nb = 1;
        int tok = -1, len = 0;
        if (M > 0 && a >= 0 && C >= 0 && M % nb == 0) {
            const int kb = M / nb, g = a - (C - nb);
            if (g >= 0 && g < nb) {
                len = kb;
                if (kb > p.max_kb) { len = 0; if (u == 0) atomicOr(p.status, FD_DEV_BAD_LENGTHS); }
                else if (u < kb) tok = p.mask_tokens[m0[b] + g * kb + u];
            }
        }
        p.next_draft[e] = tok;
        if (u == 0) p.next_len[b] = len;
    }
}

void launch_select_branch(const SelectParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    select_branch_kernel<<<1, 256, (p.batch + 1) * sizeof(int), s>>>(p);
}

}  // namespace fd
