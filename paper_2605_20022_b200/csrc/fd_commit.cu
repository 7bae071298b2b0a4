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

}  // namespace fd
