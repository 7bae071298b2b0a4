// Plan (work list of the split-KV attention) and split merge.
//
// The attention of one call is cut into tiles of 128 KV tokens.  Tiles are numbered
// sequence-major, then kv-head, then position, and the numbered list is cut into one
// contiguous range per CTA of the attention grid ("stream-K"), so every CTA streams the
// same number of KV bytes whatever the mix of prefix lengths.  A (sequence, kv-head)
// segment that falls into several ranges leaves one partial result per range; the merge
// kernel combines them in range order, which makes the result independent of timing.
//
// Ranges are cut by cost, not by tile count: a segment costs its tiles plus a fixed number of tile
// equivalents for starting it (Q load, pipeline fill and drain, epilogue), so a CTA whose range holds
// many short segments gets fewer tiles.
//
// The plan kernel checks the lengths (O(B) work, one CTA).  Page ids are checked where they are
// used, by the attention kernels: a sequence with an id outside the pool is flagged in seq_bad,
// read from page 0 instead, and has its output rows zeroed by the merge kernel.
#include <algorithm>

#include "fd_internal.cuh"

namespace fd {

// Inclusive scan of (a, b) pairs over the 256 threads of the CTA; returns the totals in (ta, tb).
__device__ inline void block_scan2(int& a, int& b, int& ta, int& tb, int (*wsum)[2]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int ua = __shfl_up_sync(0xffffffffu, a, o), ub = __shfl_up_sync(0xffffffffu, b, o);
        if (lane >= o) { a += ua; b += ub; }
    }
    __syncthreads();  // wsum may still be read from the previous round
    if (lane == 31) { wsum[warp][0] = a; wsum[warp][1] = b; }
    __syncthreads();
    int oa = 0, ob = 0;
    ta = tb = 0;
    for (int w = 0; w < 8; ++w) {
        if (w < warp) { oa += wsum[w][0]; ob += wsum[w][1]; }
        ta += wsum[w][0];
        tb += wsum[w][1];
    }
    a += oa;
    b += ob;
}

__global__ void __launch_bounds__(256) plan_kernel(AttnParams p) {
    __shared__ int s_fatal;
    __shared__ int wsum[8][2];
    // copies of the two scans the range search needs, so that its dependent probes are not global loads
    constexpr int kCache = 1024;
    __shared__ int s_ct[kCache + 1], s_ne[kCache + 1];
    // let the attention kernel behind us start its set-up now; it waits for our completion before it reads the plan
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int B = p.batch, tid = threadIdx.x;
    if (tid == 0) s_fatal = 0;
    __syncthreads();
    const int P = 16;
    long long rows = 0, tiles = 0;  // running totals over row blocks (identical in every thread)
    int nonempty = 0;               // row blocks with at least one tile so far
    // one 256-wide step of the scans the attention kernels index by: row block v has q block rows and t tiles
    auto scan_step = [&](int v, bool live, int q, int t) {
        int ne = t > 0, dummy = 0, tq, tt, tne, td;
        block_scan2(q, t, tq, tt, wsum);
        block_scan2(ne, dummy, tne, td, wsum);
        if (live) {
            p.plan.cu_q[v + 1] = (int)min(rows + q, (long long)0x7fffffff);
            p.plan.cu_tiles[v + 1] = (int)min(tiles + t, (long long)0x7fffffff);
            p.plan.cu_ne[v + 1] = nonempty + ne;
            if (v < kCache) { s_ct[v + 1] = (int)min(tiles + t, (long long)0x7fffffff); s_ne[v + 1] = nonempty + ne; }
        }
        rows += tq;
        tiles += tt;
        nonempty += tne;
    };
    // ---- pass 1, over sequences: check the lengths, cut every query block into row blocks
    const bool one_each = p.rb_per_seq == 1;  // no block is longer than a row block: sequence b is row block b, one pass
    int n_rb = 0;  // running total (identical in every thread)
    for (int base = 0; base < B; base += blockDim.x) {
        const int b = base + tid;
        int cnt = 0, dummy = 0, tc, td;
        long long n = 0, Lq = 0, M = 0, nb = 1;
        if (b < B) {
            n = p.prefix_lens[b]; Lq = p.q_lens[b]; M = p.n_mask[b];
            nb = p.n_blocks ? p.n_blocks[b] : 1;
            bool bad = n < 0 || Lq < 0 || M < 0 || M > Lq || Lq > p.max_q_len || n + Lq > (long long)p.max_pages * P;
            // several mask blocks: equal sizes, and one hypothesis (a candidate row) per block
            bad = bad || nb < 0 || (nb > 1 && (M % nb != 0 || nb > Lq - M));
            if (bad) { atomicOr(&s_fatal, 1); Lq = 0; }
            cnt = Lq > 0 ? (int)((Lq + p.rb_rows - 1) / p.rb_rows) : 1;  // an empty sequence keeps one (empty) row block
        }
        if (one_each) {
            if (b < B) {
                RowBlock rb = {b, 0, (int)n, (int)Lq, (int)M, (int)nb, {0, 0}};
                p.plan.rb[b] = rb;
            }
            scan_step(b, b < B, (int)Lq, Lq > 0 ? (int)((n + Lq + kTileTokens - 1) / kTileTokens) : 0);
            n_rb = B;
            continue;
        }
        const int mine = cnt;
        block_scan2(cnt, dummy, tc, td, wsum);
        if (b < B) {
            const int v0 = n_rb + cnt - mine;
            for (int j = 0; j < mine && v0 + j < p.max_rb; ++j) {
                RowBlock rb = {b, j * p.rb_rows, (int)n, (int)Lq, (int)M, (int)nb, {0, 0}};
                p.plan.rb[v0 + j] = rb;
            }
        }
        n_rb += tc;
    }
    if (n_rb > p.max_rb) { if (tid == 0) atomicOr(&s_fatal, 1); n_rb = p.max_rb; }
    __syncthreads();
    for (int i = tid; i < 2 * n_rb * p.Hkv; i += blockDim.x) p.plan.seg_count[i] = 0;
    // ---- pass 2, over row blocks (only where some block was cut)
    for (int base = 0; base < n_rb && !one_each; base += blockDim.x) {
        const int v = base + tid;
        int q = 0, t = 0;
        if (v < n_rb) {
            const RowBlock rb = p.plan.rb[v];
            q = max(0, min(p.rb_rows, rb.Lq - rb.i0));
            t = q > 0 ? (int)(((long long)rb.n + rb.Lq + kTileTokens - 1) / kTileTokens) : 0;
        }
        scan_step(v, v < n_rb, q, t);
    }
    if (tid == 0) { p.plan.cu_tiles[0] = 0; p.plan.cu_ne[0] = 0; s_ct[0] = 0; s_ne[0] = 0; }
    __syncthreads();
    const bool cached = n_rb <= kCache;
    auto ct_at = [&](int b) -> long long { return cached ? s_ct[b] : __ldcg(p.plan.cu_tiles + b); };
    auto ne_at = [&](int b) -> long long { return cached ? s_ne[b] : __ldcg(p.plan.cu_ne + b); };
    // Where each attention CTA starts (range_cut): a small call is not spread over every CTA -- a range is
    // worth starting only for a few tiles of work, and every extra range of a segment is one more partial to merge.
    const long long total = tiles * p.Hkv;
    const long long k = p.piece_cost;
    const long long W = (long long)p.Hkv * (tiles + k * nonempty);
    const int n_use = ranges_in_use(W, k, p.min_range_tiles, p.n_ctas);
    if (!s_fatal && total > 0 && total <= 0x7fffffffLL) {
        for (int c = tid; c <= p.n_ctas; c += blockDim.x) {
            if (c >= n_use) { p.plan.cta_start[c] = (int)total; if (c < p.n_ctas) p.plan.cta_first[c] = 0; continue; }
            int lo;
            p.plan.cta_start[c] = range_cut(c, n_use, W, n_rb, p.Hkv, k, ct_at, ne_at, &lo);
            p.plan.cta_first[c] = lo;
        }
    }
    if (tid == 0) {
        const int fatal = s_fatal || rows != p.total_q_rows || tiles * p.Hkv > 0x7fffffffLL;
        p.plan.cu_q[0] = 0;
        if (fatal) atomicOr(p.status, FD_DEV_BAD_LENGTHS);
        p.plan.hdr->fatal = fatal;
        p.plan.hdr->total_tiles = fatal ? 0 : (int)(tiles * p.Hkv);
        p.plan.hdr->n_rb = n_rb;
    }
}

void launch_plan(const AttnParams& p, cudaStream_t s) { plan_kernel<<<1, 256, 0, s>>>(p); }

// Separate merge pass (used with the SIMT attention kernel; the tensor-core kernel merges inside
// its own epilogue).  One CTA per (sequence, kv-head) segment; thread (r, cg) owns query row
// r = tid % 128 and a quarter of the columns, so partial reads are coalesced and plentiful.
constexpr int kMergeThreads = 4 * kMaxRows;

template <int D>
__global__ void __launch_bounds__(kMergeThreads) merge_kernel(AttnParams p) {
    const PlanHeader hdr = *p.plan.hdr;
    if (hdr.fatal) {  // defined output for an undefined request: zeros
        const long long n16 = (long long)p.total_q_rows * p.Hq * D / 8;
        uint4* o = reinterpret_cast<uint4*>(p.out);
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n16;
             i += (long long)gridDim.x * blockDim.x)
            o[i] = make_uint4(0, 0, 0, 0);
        return;
    }
    const int v = blockIdx.x / p.Hkv, kvh = blockIdx.x % p.Hkv;
    if (v >= hdr.n_rb) return;
    const int rows = (p.plan.cu_q[v + 1] - p.plan.cu_q[v]) * p.G;
    const int r = threadIdx.x % kMaxRows, cg = threadIdx.x / kMaxRows;
    if (r >= rows) return;
    const int ntiles = p.plan.cu_tiles[v + 1] - p.plan.cu_tiles[v];
    if (ntiles == 0) return;
    const int b = p.plan.rb[v].b;
    const int t0 = p.Hkv * p.plan.cu_tiles[v] + kvh * ntiles, t1 = t0 + ntiles;
    CtaStarts cs = {};
    cs.g = p.plan.cta_start;
    const int c_first = range_owner(cs.g, p.n_ctas, t0), c_last = range_owner(cs.g, p.n_ctas, t1 - 1);
    // an unsplit segment was written by the attention kernel itself; it is revisited only to zero it
    if (segment_pieces(cs, c_first, c_last, t0, t1) <= 1 && !sequence_flagged(p, b)) return;
    merge_row<D, D / 4>(p, cs, c_first, c_last, b, kvh, p.plan.cu_q[v], t0, t1, r, cg);
}

void launch_merge(const AttnParams& p, cudaStream_t s) {
    // the number of row blocks is known on the device only: surplus CTAs leave at once
    const int grid = (int)std::min<long long>((long long)p.batch * p.rb_per_seq, p.max_rb) * p.Hkv;
    if (grid == 0) return;
    if (p.d == 64) merge_kernel<64><<<grid, kMergeThreads, 0, s>>>(p);
    else merge_kernel<128><<<grid, kMergeThreads, 0, s>>>(p);
}

}  // namespace fd
