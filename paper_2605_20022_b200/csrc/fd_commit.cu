// KV commit / rollback: length truncation and page release, one CTA.
#include "fd_internal.cuh"

namespace fd {

__global__ void __launch_bounds__(256) commit_kernel(CommitParams p) {
    extern __shared__ int s_off[];  // [B+1] exclusive scan of pages freed per sequence
    const int tid = threadIdx.x, P = p.page_size;
    for (int b = tid; b < p.batch; b += blockDim.x) {
        const int a = p.accepted[b], Lq = p.q_lens[b], n = p.prefix_lens[b];
        int cnt = 0;
        if (a >= 0) {
            if (a >= Lq || Lq < 0 || n < 0 || (long long)n + Lq > (long long)p.max_pages * P) {
                atomicOr(p.status, FD_DEV_BAD_ACCEPT);
                cnt = -1;  // marks "leave unchanged"
            } else {
                cnt = (n + Lq + P - 1) / P - (n + a + 1 + P - 1) / P;
            }
        }
        s_off[b + 1] = cnt;
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        s_off[0] = 0;
        for (int b = 0; b < p.batch; ++b) {
            const int cnt = s_off[b + 1];
            s_off[b + 1] = (cnt < 0) ? -(run + 1) : run + cnt;  // negative = skip, still carries the offset
            run += max(cnt, 0);
        }
        *p.n_freed = run;
    }
    __syncthreads();
    for (int b = tid; b < p.batch; b += blockDim.x) {
        const int a = p.accepted[b];
        if (a < 0 || s_off[b + 1] < 0) continue;
        int prev = s_off[b];
        if (prev < 0) prev = -prev - 1;
        const int n = p.prefix_lens[b], new_len = n + a + 1;
        const int keep = (new_len + P - 1) / P, old_pages = (n + p.q_lens[b] + P - 1) / P;
        int32_t* row = p.page_table + (long long)b * p.max_pages;
        for (int pg = keep; pg < old_pages; ++pg) {
            p.freed[prev + (pg - keep)] = row[pg];
            row[pg] = -1;
        }
        p.prefix_lens[b] = new_len;
    }
}

void launch_commit(const CommitParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    commit_kernel<<<1, 256, (p.batch + 1) * sizeof(int), s>>>(p);
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
