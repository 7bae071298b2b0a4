// Verification by speculative sampling (temperature > 0): accept each draft with probability
// min(1, p(x) / q(x)), draw the bonus token from the residual max(0, p - q) at the first rejection, or from
// p after the last draft when everything was accepted.  p = softmax(target logits / T), q = softmax(draft
// logits / T), or all mass on the proposed token when no draft logits are given.  The uniforms are inputs.
//
// Two sweeps, both made of 4096-logit chunks:
//   stats   one CTA per (candidate row, chunk): chunk maximum and sum exp((x - max) / T) of the target row
//           and of the draft row.  The CTA that delivers a row's last chunk folds them into the row's
//           (max, Z); the CTA that finishes last of all runs the accept test of every sequence -- it needs
//           p(x) and q(x) of single tokens only -- and notes which row each bonus token is drawn from.
//   sample  one CTA per (sequence, chunk): sum of the chunk's weights w(y) (p, p without x, or the clipped
//           difference).  The CTA that delivers a sequence's last chunk inverts the cumulative sum in index
//           order: it finds the chunk in which u * total is crossed, recomputes that chunk and finds the token.
// Every reduction has a fixed order, so results do not depend on timing.
#include "fd_internal.cuh"

namespace fd {

namespace {

constexpr int kVec = kAcceptChunk / (4 * 256);  // float4 per thread and chunk

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Loads this thread's 4 * kVec logits of chunk [c0, c0 + n) of `row_ptr`; -inf past the end.
__device__ __forceinline__ void load_chunk(const float* base, int n, int tid, float (&x)[4 * kVec]) {
    const bool vec = (reinterpret_cast<uintptr_t>(base) & 15) == 0;
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        const int e = 4 * (tid + k * 256);
        if (vec && e + 3 < n) {
            const float4 a = __ldcs(reinterpret_cast<const float4*>(base + e));
            x[4 * k] = a.x; x[4 * k + 1] = a.y; x[4 * k + 2] = a.z; x[4 * k + 3] = a.w;
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) x[4 * k + q] = (e + q < n) ? base[e + q] : -INFINITY;
        }
    }
}

// Block-wide sum over 256 threads in a fixed order; every thread gets the result.
__device__ __forceinline__ float block_sum(float v, float* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) r += sh[w];
    return r;
}

// (max, sum exp((x - max) * kt)) of this CTA's chunk: every warp reduces its own share to (max, sum) with
// shuffles, thread 0 folds the eight pairs in warp order -- one barrier, fixed order.  `sh` holds 8 float2.
__device__ __forceinline__ void warp_stats(const float (&x)[4 * kVec], float kt, float2* sh) {
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < 4 * kVec; ++k) m = fmaxf(m, x[k]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float s = 0.f;
    if (m > -INFINITY) {  // a warp whose share lies wholly past the end of the row has nothing
        const float nm = -m * kt;
#pragma unroll
        for (int k = 0; k < 4 * kVec; ++k) s += ex2f(fmaf(x[k], kt, nm));  // one FMA per element; -inf padding adds 0
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = make_float2(m, s);
}
__device__ __forceinline__ float2 fold_stats(const float2* sh, float kt) {
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < 8; ++w) m = fmaxf(m, sh[w].x);
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w)
        if (sh[w].x > -INFINITY) s += sh[w].y * ex2f((sh[w].x - m) * kt);
    return make_float2(m, s);
}

// Warps 0 and 1 of the CTA that delivered the last chunk of `row` fold the row's chunk partials into (max, Z).
__device__ __forceinline__ void sv_finish_row(const SampleParams& p, int row, int chunks) {
    const int tid = threadIdx.x;
    if (tid < 64) {  // warp 0: target row, warp 1: draft row
        __threadfence();
        const int which = tid >> 5;
        // the partials of a row are interleaved (target, draft): view one of them with stride 2
        const float2* part = p.part + (long long)row * chunks * 2 + which;
        float m = -INFINITY;
        for (int c = (tid & 31); c < chunks; c += 32) m = fmaxf(m, __ldcg(&part[2 * c].x));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float z = 0.f;
        for (int c = (tid & 31); c < chunks; c += 32) {
            const float2 v = __ldcg(part + 2 * c);
            z += v.y * ex2f((v.x - m) * p.kt);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
        if ((tid & 31) == 0) {
            p.row_stat[2 * row + which] = make_float2(m, z);
            if (which == 0) p.row_ticket[row] = 0u;
        }
    }
}

// The CTA that finished last of all: accept tests, accepted lengths, and which row each bonus token is drawn from.
__device__ __forceinline__ void sv_final(const SampleParams& p) {
    const int tid = threadIdx.x;
    // ---- one CTA.  First the accept test of every row against the draft fed at the next row, all rows in
    //      parallel (each test reads single logits that no cache holds); a sequence's last row has no draft
    //      to test and its flag is never looked at.
    for (int r = tid; r < p.total_rows; r += blockDim.x) {
        bool okf = false;
        const int xt = r + 1 < p.total_rows ? p.drafts[r + 1] : -1;
        if ((unsigned)xt < (unsigned)p.vocab) {  // anything else is not a token and cannot be accepted
            const float2 ts = __ldcg(p.row_stat + 2 * r);
            const float px = ex2f((p.logits[(long long)r * p.vocab + xt] - ts.x) * p.kt) / ts.y;
            float qx = 1.f;
            if (p.draft_logits) {
                const float2 ds = __ldcg(p.row_stat + 2 * r + 1);
                qx = ex2f((p.draft_logits[(long long)r * p.vocab + xt] - ds.x) * p.kt) / ds.y;
            }
            okf = p.u_accept[r] * qx < px;  // u < min(1, p / q), with u < 1
        }
        p.flags[r] = okf ? 1 : 0;
    }
    // ---- then a thread per sequence: first candidate row by a scan, accepted length = leading passes
    __shared__ int carry, wcnt[8], s_bad;
    if (tid == 0) { carry = 0; s_bad = 0; }
    __syncthreads();
    for (int base = 0; base < p.batch; base += blockDim.x) {
        const int b = base + tid;
        int C = 0;
        if (b < p.batch) {
            C = p.q_lens[b] - p.n_mask[b];
            if (C < 0 || p.n_mask[b] < 0) { atomicOr(&s_bad, 1); C = 0; }
        }
        int inc = C;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, inc, o);
            if ((tid & 31) >= o) inc += u;
        }
        if ((tid & 31) == 31) wcnt[tid >> 5] = inc;
        __syncthreads();
        long long offr = carry;
        for (int w = 0; w < (tid >> 5); ++w) offr += wcnt[w];
        const long long r0 = offr + inc - C;
        if (b < p.batch) {
            int a = -1, srow = -1, mode = 0, xs = -1;
            if (C > 0 && r0 + C <= p.total_rows) {
                const int k = C - 1;
                a = 0;
                while (a < k && p.flags[r0 + a]) ++a;
                if (a < k) xs = p.drafts[r0 + a + 1];
                srow = (int)(r0 + a);
                mode = (a == k) ? 0 : (p.draft_logits ? 1 : 2);
                if (mode == 2 && (unsigned)xs >= (unsigned)p.vocab) mode = 0;  // nothing to take out of p
            }
            p.accepted[b] = a;
            if (a < 0) p.bonus[b] = -1;
            p.seq_info[b] = make_int4(srow, mode, xs, 0);
        }
        __syncthreads();
        if (tid == blockDim.x - 1) carry = (int)min(offr + inc, (long long)0x7fffffff);
        __syncthreads();
    }
    // lengths that do not add up: a defined output, -1 everywhere, and nothing for the draw kernel to do
    const bool bad = s_bad || carry != p.total_rows;  // final after the loop's last barrier
    if (bad) {
        for (int b = tid; b < p.batch; b += blockDim.x) {
            p.accepted[b] = -1;
            p.bonus[b] = -1;
            p.seq_info[b] = make_int4(-1, 0, -1, 0);
        }
    }
    if (tid == 0) {
        if (bad) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
        *p.ticket = 0u;
    }
}

__global__ void __launch_bounds__(256) sv_stats_kernel(SampleParams p, int chunks) {
    __shared__ float2 sh_t[8], sh_d[8];
    __shared__ bool row_last, last;
    const int row = blockIdx.x / chunks, chunk = blockIdx.x % chunks, tid = threadIdx.x;
    const int c0 = chunk * kAcceptChunk, n = min(p.vocab, c0 + kAcceptChunk) - c0;
    const long long off = (long long)row * p.vocab + c0;
    float x[4 * kVec], d[4 * kVec];
    load_chunk(p.logits + off, n, tid, x);                        // both rows' loads are in flight together
    if (p.draft_logits) load_chunk(p.draft_logits + off, n, tid, d);
    warp_stats(x, p.kt, sh_t);
    if (p.draft_logits) warp_stats(d, p.kt, sh_d);
    __syncthreads();
    if (tid == 0) {
        p.part[((long long)row * chunks + chunk) * 2] = fold_stats(sh_t, p.kt);
        p.part[((long long)row * chunks + chunk) * 2 + 1] = p.draft_logits ? fold_stats(sh_d, p.kt) : make_float2(0.f, 1.f);
        __threadfence();
        row_last = atomicAdd(p.row_ticket + row, 1u) == (unsigned)chunks - 1;
    }
    __syncthreads();
    if (!row_last) return;  // only the CTA that completes a row goes on: one fence + count per chunk, not two
    sv_finish_row(p, row, chunks);
    __syncthreads();
    if (tid == 0) {  // rows completed so far: whoever completes the last row finishes the call
        __threadfence();
        last = atomicAdd(p.ticket, 1u) == (unsigned)p.total_rows - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    // (behind an attention call the sweep has not waited for it; this one CTA does, before the results are written)
    if (p.chained) asm volatile("griddepcontrol.wait;" ::: "memory");
    sv_final(p);
}

// Weight of token y in the distribution the bonus token is drawn from.  ts / ds: (row maximum, 1 / Z) of the target
// and of the draft row.
__device__ __forceinline__ float weight(float lt, float ld, int y, int mode, int xs, float2 ts, float2 ds, float kt) {
    const float pv = ex2f((lt - ts.x) * kt) * ts.y;
    if (mode == 0) return pv;
    if (mode == 2) return y == xs ? 0.f : pv;
    return fmaxf(pv - ex2f((ld - ds.x) * kt) * ds.y, 0.f);
}

__global__ void __launch_bounds__(256) sv_sample_kernel(SampleParams p, int chunks) {
    __shared__ float sh[8];
    __shared__ bool seq_last;
    __shared__ int s_chunk;
    __shared__ float s_before;
    const int b = blockIdx.x / chunks, chunk = blockIdx.x % chunks, tid = threadIdx.x;
    const int4 info = p.seq_info[b];
    const int row = info.x, mode = info.y, xs = info.z;
    if (row < 0) return;  // uniform: no candidate rows, outputs already written
    float2 ts = p.row_stat[2 * row], ds = p.row_stat[2 * row + 1];
    ts.y = 1.f / ts.y;  // the weights multiply by 1 / Z
    ds.y = 1.f / ds.y;
    {
        const int c0 = chunk * kAcceptChunk, n = min(p.vocab, c0 + kAcceptChunk) - c0;
        const long long off = (long long)row * p.vocab + c0;
        float x[4 * kVec], d[4 * kVec];
        load_chunk(p.logits + off, n, tid, x);
        if (mode == 1) load_chunk(p.draft_logits + off, n, tid, d);
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < kVec; ++k)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int e = 4 * (tid + k * 256) + q;
                if (e < n) s += weight(x[4 * k + q], mode == 1 ? d[4 * k + q] : 0.f, c0 + e, mode, xs, ts, ds, p.kt);
            }
        s = block_sum(s, sh);
        if (tid == 0) {
            p.chunk_w[(long long)b * chunks + chunk] = s;
            __threadfence();
            seq_last = atomicAdd(p.seq_ticket + b, 1u) == (unsigned)chunks - 1;
        }
    }
    __syncthreads();
    if (!seq_last) return;
    __threadfence();
    // ---- the chunk in which the cumulative weight passes u * total: warp 0, a lane per chunk (32 at a time), the
    //      running sums by a shuffle scan in chunk order, so that the loads of a group are one round trip
    if (tid < 32) {
        const float* cw = p.chunk_w + (long long)b * chunks;
        float total = 0.f;  // identical in every lane
        for (int base = 0; base < chunks; base += 32) {
            float v = base + tid < chunks ? __ldcg(cw + base + tid) : 0.f;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float u = __shfl_up_sync(0xffffffffu, v, o);
                if (tid >= o) v += u;
            }
            total += __shfl_sync(0xffffffffu, v, 31);
        }
        const float target = p.u_bonus[b] * total;
        int pick = -1, last_pos = 0;
        float before = 0.f, carry = 0.f, last_before = 0.f;
        for (int base = 0; base < chunks && pick < 0; base += 32) {
            const float wc = base + tid < chunks ? __ldcg(cw + base + tid) : 0.f;
            float inc = wc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float u = __shfl_up_sync(0xffffffffu, inc, o);
                if (tid >= o) inc += u;
            }
            const float cum_before = carry + inc - wc;           // weight of the chunks before this lane's
            const unsigned hit = __ballot_sync(0xffffffffu, wc > 0.f && cum_before + wc > target);
            const unsigned pos = __ballot_sync(0xffffffffu, wc > 0.f);
            if (pos) {
                const int lp = 31 - __clz(pos);
                last_pos = base + lp;
                last_before = __shfl_sync(0xffffffffu, cum_before, lp);
            }
            if (hit) {
                const int first = __ffs(hit) - 1;
                pick = base + first;
                before = __shfl_sync(0xffffffffu, cum_before, first);
            }
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (pick < 0) { pick = last_pos; before = last_before; }  // rounding left the target at or past the total
        if (tid == 0) {
            s_chunk = pick;
            s_before = target - before;  // what is left to cross inside the chunk
            p.seq_ticket[b] = 0u;
        }
    }
    __syncthreads();
    // ---- inside the chunk: thread t owns 16 consecutive tokens; exclusive scan of the thread sums, in order
    const int c0 = s_chunk * kAcceptChunk, n = min(p.vocab, c0 + kAcceptChunk) - c0;
    const float rest = s_before;
    const long long off = (long long)row * p.vocab + c0;
    constexpr int kPer = kAcceptChunk / 256;
    float w[kPer];
    float mine = 0.f;
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int e = tid * kPer + k;
        w[k] = 0.f;
        if (e < n) w[k] = weight(p.logits[off + e], mode == 1 ? p.draft_logits[off + e] : 0.f, c0 + e, mode, xs, ts, ds, p.kt);
        mine += w[k];
    }
    __shared__ float wsum[8];
    __shared__ int s_tok, s_lastpos;
    float inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float u = __shfl_up_sync(0xffffffffu, inc, o);
        if ((tid & 31) >= o) inc += u;
    }
    if (tid == 0) { s_tok = 0x7fffffff; s_lastpos = -1; }
    if ((tid & 31) == 31) wsum[tid >> 5] = inc;
    __syncthreads();
    float excl = inc - mine;
    for (int wv = 0; wv < (tid >> 5); ++wv) excl += wsum[wv];
    // first token whose inclusive cumulative weight exceeds `rest`
    float cum = excl;
    int found = 0x7fffffff, lastpos = -1;
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        if (w[k] > 0.f) lastpos = c0 + tid * kPer + k;
        cum += w[k];
        if (found == 0x7fffffff && w[k] > 0.f && cum > rest) found = c0 + tid * kPer + k;
    }
    if (found != 0x7fffffff) atomicMin(&s_tok, found);
    if (lastpos >= 0) atomicMax(&s_lastpos, lastpos);
    __syncthreads();
    if (tid == 0) p.bonus[b] = s_tok != 0x7fffffff ? s_tok : max(s_lastpos, 0);
}

__global__ void sv_empty_kernel(SampleParams p) {
    for (int b = threadIdx.x; b < p.batch; b += blockDim.x) {
        if (p.q_lens[b] - p.n_mask[b] != 0) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
        p.accepted[b] = -1;
        p.bonus[b] = -1;
    }
}

}  // namespace

int launch_accept_sample(const SampleParams& p, cudaStream_t s) {
    if (p.batch == 0) return 0;
    if (p.total_rows == 0) { sv_empty_kernel<<<1, 256, 0, s>>>(p); return 1; }
    const int chunks = (p.vocab + kAcceptChunk - 1) / kAcceptChunk;
    if (!p.chained) {
        sv_stats_kernel<<<p.total_rows * chunks, 256, 0, s>>>(p, chunks);
    } else {
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(p.total_rows * chunks);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = s;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, sv_stats_kernel, p, chunks);
}
    sv_sample_kernel<<<p.batch * chunks, 256, 0, s>>>(p, chunks);
    return 2;
}

}  // namespace fd
