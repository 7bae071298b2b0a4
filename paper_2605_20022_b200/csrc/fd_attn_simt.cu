// CUDA-core split-KV attention under the hybrid mask: the general-shape path.
//
// One thread owns one query row of a (sequence, kv-head) segment -- row r = i * G + g is
// block row i of q-head kvh * G + g -- so the G q-heads of a kv-head and all rows of the
// query block share every KV page that is brought into shared memory.  The mask is never
// materialised: a row carries the first key position it may NOT see (`limit`), which is
// n + i + 1 for a candidate row (causal, no mask token) and kv_len for a mask row (prefix,
// candidates, whole mask block).  Softmax is the online form in the log2 domain.
#include "fd_internal.cuh"

namespace fd {

template <int D>
__device__ inline void store_out_row(__nv_bfloat16* dst, const float* o, float inv) {
#pragma unroll
    for (int c = 0; c < D; c += 8) {
        __align__(16) __nv_bfloat162 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = __floats2bfloat162_rn(o[c + 2 * k] * inv, o[c + 2 * k + 1] * inv);
        *reinterpret_cast<uint4*>(dst + c) = *reinterpret_cast<const uint4*>(v);
    }
}

template <int D>
__global__ void __launch_bounds__(kMaxRows) attn_simt_kernel(AttnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* qT = reinterpret_cast<float*>(smem_raw);                                   // [D][128], pre-scaled
    __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(smem_raw + D * kMaxRows * 4);  // [16][D]
    __nv_bfloat16* vs = ks + 16 * D;                                                  // [16][D]

    const PlanHeader hdr = *p.plan.hdr;
    const int total = hdr.total_tiles;
    if (total == 0) return;
    const int cta = blockIdx.x, r = threadIdx.x;
    const int s_c = p.plan.cta_start[cta], e_c = p.plan.cta_start[cta + 1];

    int t = s_c;
    while (t < e_c) {
        // row block that owns tile t: last v with Hkv * cu_tiles[v] <= t
        int lo = 0, hi = hdr.n_rb;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.Hkv * p.plan.cu_tiles[mid] <= t) lo = mid; else hi = mid;
        }
        const int v = lo;
        const RowBlock rb = p.plan.rb[v];
        const int b = rb.b;
        const int ntiles = p.plan.cu_tiles[v + 1] - p.plan.cu_tiles[v];
        const int rem = t - p.Hkv * p.plan.cu_tiles[v];
        const int kvh = rem / ntiles, tile0 = rem % ntiles;
        const int seg_start = t - tile0, seg_end = seg_start + ntiles;
        const int t_end = min(e_c, seg_end);
        const int n = rb.n, Lq = rb.Lq, M = rb.M;
        const int kv_len = n + Lq, rows = min(p.rb_rows, Lq - rb.i0) * p.G, row0 = p.plan.cu_q[v];
        const int i = r / p.G, g = r % p.G;
        const RowMask rm = row_mask(rb.i0 + i, n, Lq, M, rb.nb, r < rows);

        __syncthreads();  // previous piece is done with qT
        if (r < rows) {
            const __nv_bfloat16* qr = p.q + ((long long)(row0 + i) * p.Hq + kvh * p.G + g) * D;
#pragma unroll 4
            for (int c = 0; c < D; c += 8) {
                const uint4 raw = *reinterpret_cast<const uint4*>(qr + c);
                const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
                for (int k = 0; k < 8; ++k) qT[(c + k) * kMaxRows + r] = __bfloat162float(e[k]) * p.scale_log2e;
            }
        } else {
            for (int c = 0; c < D; ++c) qT[c * kMaxRows + r] = 0.f;
        }

        float m = -INFINITY, l = 0.f, acc[D];
#pragma unroll
        for (int c = 0; c < D; ++c) acc[c] = 0.f;

        for (int tile = tile0; tile < tile0 + (t_end - t); ++tile) {
            for (int pg = 0; pg < kTileTokens / 16; ++pg) {
                const int pos0 = tile * kTileTokens + pg * 16;
                if (pos0 >= kv_len) break;
                int phys = p.page_table[(long long)b * p.max_pages + pos0 / 16];
                if ((unsigned)phys >= (unsigned)p.num_pages) {  // never form an address from a bad id
                    if (r == 0) flag_sequence(p, b);
                    phys = 0;
                }
                const __nv_bfloat16* kp = p.kv + (((long long)phys * 2 + 0) * p.Hkv + kvh) * 16 * D;
                const __nv_bfloat16* vp = p.kv + (((long long)phys * 2 + 1) * p.Hkv + kvh) * 16 * D;
                __syncthreads();  // everyone is done with the previous page
                for (int e = r; e < 16 * D / 8; e += kMaxRows) {
                    reinterpret_cast<uint4*>(ks)[e] = reinterpret_cast<const uint4*>(kp)[e];
                    reinterpret_cast<uint4*>(vs)[e] = reinterpret_cast<const uint4*>(vp)[e];
                }
                __syncthreads();
                if (r >= rows) continue;
                // keys of this page the row may see (bit k = token k); none -> nothing to do for this row
                unsigned vis = 0;
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int j = pos0 + k;
                    if (j < kv_len && (j < rm.limit || (j >= rm.blk_lo && j < rm.blk_hi))) vis |= 1u << k;
                }
                if (vis == 0) continue;
                float s[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) s[k] = 0.f;
                for (int c = 0; c < D; c += 2) {
                    const float q0 = qT[c * kMaxRows + r], q1 = qT[(c + 1) * kMaxRows + r];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const float2 kk = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(ks + k * D + c));
                        s[k] = fmaf(q0, kk.x, fmaf(q1, kk.y, s[k]));
                    }
                }
                float pm = -INFINITY;
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    s[k] = ((vis >> k) & 1u) ? s[k] : -INFINITY;  // a select, never a multiply: hidden slots may hold NaN
                    pm = fmaxf(pm, s[k]);
                }
                const float m_new = fmaxf(m, pm);
                const float alpha = (m == -INFINITY) ? 0.f : exp2f(m - m_new);
                l *= alpha;
#pragma unroll
                for (int c = 0; c < D; ++c) acc[c] *= alpha;
                m = m_new;
#pragma unroll 1
                for (int k = 0; k < 16; ++k) {
                    if (!((vis >> k) & 1u)) continue;
                    const float pj = exp2f(s[k] - m);
                    l += pj;
#pragma unroll
                    for (int c = 0; c < D; c += 2) {
                        const float2 vv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(vs + k * D + c));
                        acc[c] = fmaf(pj, vv.x, acc[c]);
                        acc[c + 1] = fmaf(pj, vv.y, acc[c + 1]);
                    }
                }
            }
        }

        const bool complete = (t == seg_start) && (t_end == seg_end);
        if (r < rows) {
            if (complete) {
                store_out_row<D>(p.out + ((long long)(row0 + i) * p.Hq + kvh * p.G + g) * D, acc, 1.f / l);
            } else {
                const int slot = 2 * cta + (t == s_c ? 0 : 1);
                p.part.m[slot * kMaxRows + r] = m;
                p.part.l[slot * kMaxRows + r] = l;
                float4* o = partial_o4(p.part, D, slot, 0, r);
#pragma unroll
                for (int c = 0; c < D; c += 4) o[(c >> 2) * kMaxRows] = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
            }
        }
        t = t_end;
    }
}

// 66 KB + 8 KB of dynamic shared memory needs the opt-in; a per-device attribute, set once per context at fd_create.
cudaError_t attn_simt_prepare(int d) {
    if (d != 128) return cudaSuccess;
    return cudaFuncSetAttribute(attn_simt_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * kMaxRows * 4 + 2 * 16 * 128 * 2);
}

void launch_attn_simt(const AttnParams& p, cudaStream_t s) {
    if (p.batch == 0) return;
    const int smem = p.d * kMaxRows * 4 + 2 * 16 * p.d * 2;
    if (p.d == 64) {
        attn_simt_kernel<64><<<p.n_ctas, kMaxRows, smem, s>>>(p);
    } else {
        attn_simt_kernel<128><<<p.n_ctas, kMaxRows, smem, s>>>(p);
    }
}

}  // namespace fd
