// C ABI of libflexdraft: context, argument checks, launch sequencing.
#include <math.h>
#include <algorithm>
#include <vector>
#include <utility>
#include <new>

#include "fd_internal.cuh"

struct fd_ctx {
    fd_config cfg;
    int device;
    int n_sms;
    int n_ctas;        // attention grid
    int attn_path;     // resolved FD_ATTN_SIMT or FD_ATTN_TCGEN05
    int tc_choice;     // FD_ATTN_TCGEN05 (per call), FD_ATTN_TCGEN05_PLANNED or FD_ATTN_TCGEN05_SELF_PLANNED
    int last_mode;     // FD_TC_* of the last tensor-core call
    int epoch;         // number of the last attention call (never 0 once a call was made)
    float scale_log2e;
    // scratch (device)
    unsigned char* pool;
    fd::Plan plan;
    fd::PartialView part;
    unsigned long long* keys;
    unsigned int* ticket;
    unsigned long long* ds_key;  // draft-select chunk partials [max_rows][chunks]
    float* ds_sum;
    unsigned int* ds_ticket;
    unsigned int* ds_row_ticket;
    float2* sv_part;             // speculative-sampling scratch
    float2* sv_row;
    unsigned int *sv_row_ticket, *sv_ticket, *sv_seq_ticket;
    int4* sv_seq;
    float* sv_chunk_w;
    unsigned char* sv_flags;
    int* status;
    int max_rows;      // capacity of keys
    int max_rb;        // capacity of the row-block arrays of the plan
    void* tc_state;
    long long launches;
    // a pinned plan: the work list of one step, reused by every attention call with these lengths
    bool pinned;
    int pin_batch, pin_rows;
    const int32_t *pin_pl, *pin_ql, *pin_nm, *pin_nb;
    bool pin_chain;    // the context's last launch was an attention or append call under the pinned plan (see AttnParams::early)
    bool chain_append; // ... and it was the append (which writes the cache the next attention call reads)
    bool after_attn;   // the context's last launch was an attention call of the tensor-core kernel (it lets its dependents in early)
    bool back_to_back; // fd_calls_back_to_back: nothing but this context's own launches sits between its calls on the stream
    std::vector<std::pair<uintptr_t, uintptr_t>> chain_out;  // [begin, end) of what the attention calls of the chain have written
    struct HostStage* host;  // staging for fd_step_host, nullptr until fd_host_reserve
};

// Device staging + copy streams of the host-buffer step (fd_host_reserve / fd_step_host).
struct HostStage {
    int max_q_rows, max_cand_rows;
    cudaStream_t h2d, d2h;
    cudaEvent_t start, meta, logits, done, fin, q_ready[2], attn_done[2], out_copied[2];
    unsigned char* pool;
    void *q[2], *out[2], *kn[2], *vn[2];
    float* lg;
    int32_t *drafts, *pt, *pl, *ql, *nm, *nb, *acc, *bon, *freed, *nfreed;
};

// Tile equivalents charged for starting a segment in a CTA's range of the tensor-core kernel (measured:
// ranges balance best when a segment start is charged about five tiles).
#ifndef FD_PIECE_COST
#define FD_PIECE_COST 5
#endif
// Least tiles for which a CTA of the tensor-core kernel gets a range of its own: a small call then runs on
// fewer CTAs, each with a few tiles, instead of one tile everywhere and many partials to merge.
#ifndef FD_MIN_RANGE_TILES
#define FD_MIN_RANGE_TILES 2
#endif

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

// The part of the attention parameters that the plan kernel needs (lengths and geometry).
static fd::AttnParams attn_params(fd_ctx* c, int batch, int total_q_rows, const int32_t* prefix_lens, const int32_t* q_lens,
                                  const int32_t* n_mask, const int32_t* n_blocks) {
    fd::AttnParams p = {};
    p.batch = batch; p.total_q_rows = total_q_rows;
    p.Hq = c->cfg.n_q_heads; p.Hkv = c->cfg.n_kv_heads; p.G = p.Hq / p.Hkv; p.d = c->cfg.head_dim;
    p.max_pages = c->cfg.max_pages_per_seq; p.max_q_len = c->cfg.max_q_len;
    p.rb_rows = fd::kMaxRows / p.G;
    p.rb_per_seq = (p.max_q_len + p.rb_rows - 1) / p.rb_rows;
    p.max_rb = c->max_rb;
    p.scale_log2e = c->scale_log2e;
    p.prefix_lens = prefix_lens; p.q_lens = q_lens; p.n_mask = n_mask; p.n_blocks = n_blocks;
    p.plan = c->plan; p.part = c->part; p.n_ctas = c->n_ctas; p.status = c->status;
    p.q_box_t = fd::q_box_rows(p.G);
    p.piece_cost = c->attn_path == FD_ATTN_SIMT ? 0 : FD_PIECE_COST;
    p.min_range_tiles = c->attn_path == FD_ATTN_SIMT ? 1 : FD_MIN_RANGE_TILES;
    return p;
}


extern "C" {

const char* fd_status_string(fd_status s) {
    switch (s) {
        case FD_OK: return "FD_OK";
        case FD_ERR_INVALID_ARG: return "FD_ERR_INVALID_ARG";
        case FD_ERR_UNSUPPORTED: return "FD_ERR_UNSUPPORTED";
        case FD_ERR_WORKSPACE: return "FD_ERR_WORKSPACE";
        case FD_ERR_CUDA: return "FD_ERR_CUDA";
        case FD_ERR_DEVICE_STATUS: return "FD_ERR_DEVICE_STATUS";
        case FD_ERR_STATIC_LIMIT: return "FD_ERR_STATIC_LIMIT";
    }
    return "FD_UNKNOWN";
}

fd_status fd_create(fd_ctx** out, const fd_config* cfg) {
    if (!out) return FD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return FD_ERR_INVALID_ARG;
    if (cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->vocab <= 0 || cfg->max_batch <= 0 ||
        cfg->max_q_len <= 0 || cfg->max_pages_per_seq <= 0 || cfg->softmax_scale < 0.f)
        return FD_ERR_INVALID_ARG;
    if (cfg->n_q_heads % cfg->n_kv_heads != 0) return FD_ERR_INVALID_ARG;
    if (cfg->attn_path < FD_ATTN_AUTO || cfg->attn_path > FD_ATTN_TCGEN05_SELF_PLANNED) return FD_ERR_INVALID_ARG;
    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    if ((cfg->head_dim != 64 && cfg->head_dim != 128) || cfg->page_size != 16) return FD_ERR_UNSUPPORTED;
    if (G > fd::kMaxRows || cfg->max_q_len > 4096) return FD_ERR_UNSUPPORTED;  // at least one block row per 128-row tile
    if ((long long)cfg->max_pages_per_seq * 16 > 0x3fffffffLL || cfg->max_batch > 4096) return FD_ERR_UNSUPPORTED;

    fd_ctx* c = new (std::nothrow) fd_ctx();
    if (!c) return FD_ERR_WORKSPACE;
    c->cfg = *cfg;
    c->launches = 0;
    c->tc_state = nullptr;
    c->host = nullptr;
    c->pinned = false;
    c->pin_chain = false;
    if (cudaGetDevice(&c->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) {
        delete c;
        return FD_ERR_CUDA;
    }
    const float scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
    c->scale_log2e = scale * 1.4426950408889634f;

    const bool tc_ok = fd::attn_tc_supported(cfg->head_dim, G, cfg->max_q_len);
    if (cfg->attn_path >= FD_ATTN_TCGEN05 && !tc_ok) { delete c; return FD_ERR_UNSUPPORTED; }
    c->tc_choice = cfg->attn_path >= FD_ATTN_TCGEN05 ? cfg->attn_path : FD_ATTN_TCGEN05;
    c->last_mode = -1;
    c->chain_append = false;
    c->after_attn = false;
    c->back_to_back = false;
    c->epoch = 0;
    c->attn_path = (cfg->attn_path == FD_ATTN_SIMT || !tc_ok) ? FD_ATTN_SIMT : FD_ATTN_TCGEN05;
    // SIMT kernel: two 74 KB CTAs fit an SM; tensor-core kernel: one persistent CTA per SM
    c->n_ctas = c->attn_path == FD_ATTN_SIMT ? 2 * c->n_sms : c->n_sms;
    if (c->attn_path == FD_ATTN_SIMT && fd::attn_simt_prepare(cfg->head_dim) != cudaSuccess) { cudaGetLastError(); delete c; return FD_ERR_CUDA; }

    const int B = cfg->max_batch, d = cfg->head_dim;
    const size_t slots = 2 * (size_t)c->n_ctas;
    c->max_rows = (int)std::min<long long>((long long)B * cfg->max_q_len, 0x7fffffffLL);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    // a query block longer than 128 / G rows is handled as several row blocks: size their arrays for the worst case
    const int rb_rows = fd::kMaxRows / G;
    c->max_rb = (int)std::min<long long>((long long)B * ((cfg->max_q_len + rb_rows - 1) / rb_rows), 0x7fffffffLL / 64);
    const size_t NR = (size_t)c->max_rb;
    const size_t o_hdr = take(sizeof(fd::PlanHeader));
    const size_t o_rb = take(NR * sizeof(fd::RowBlock));
    const size_t o_cuq = take((NR + 1) * sizeof(int));
    const size_t o_cut = take((NR + 1) * sizeof(int));
    const size_t o_ok = take(B * sizeof(int));
    const size_t o_sc = take(2 * NR * cfg->n_kv_heads * sizeof(int));
    const size_t o_cf = take((size_t)c->n_ctas * sizeof(int));
    const size_t o_cs = take(((size_t)c->n_ctas + 1) * sizeof(int));
    const size_t o_cne = take((NR + 1) * sizeof(int));
    const size_t o_po = take(slots * d * fd::kMaxRows * sizeof(float));
    const size_t o_pm = take(slots * fd::kMaxRows * sizeof(float));
    const size_t o_pl = take(slots * fd::kMaxRows * sizeof(float));
    const size_t o_keys = take((size_t)c->max_rows * sizeof(unsigned long long));
    const size_t o_tick = take(sizeof(unsigned int));
    const size_t ds_chunks = (size_t)(cfg->vocab + fd::kAcceptChunk - 1) / fd::kAcceptChunk;
    const size_t o_dsk = take((size_t)c->max_rows * ds_chunks * sizeof(unsigned long long));
    const size_t o_dss = take((size_t)c->max_rows * ds_chunks * sizeof(float));
    const size_t o_dst = take(sizeof(unsigned int));
    const size_t o_dsr = take((size_t)c->max_rows * sizeof(unsigned int));
    const size_t o_svp = take((size_t)c->max_rows * ds_chunks * 2 * sizeof(float2));
    const size_t o_svr = take((size_t)c->max_rows * 2 * sizeof(float2));
    const size_t o_svrt = take((size_t)c->max_rows * sizeof(unsigned int));
    const size_t o_svt = take(sizeof(unsigned int));
    const size_t o_svst = take((size_t)B * sizeof(unsigned int));
    const size_t o_svs = take((size_t)B * sizeof(int4));
    const size_t o_svw = take((size_t)B * ds_chunks * sizeof(float));
    const size_t o_svf = take((size_t)c->max_rows);
    const size_t o_stat = take(sizeof(int));
    if (cudaMalloc(&c->pool, off) != cudaSuccess) { cudaGetLastError(); delete c; return FD_ERR_WORKSPACE; }
    if (cudaMemset(c->pool, 0, off) != cudaSuccess) { cudaFree(c->pool); delete c; return FD_ERR_CUDA; }
    c->plan.hdr = reinterpret_cast<fd::PlanHeader*>(c->pool + o_hdr);
    c->plan.rb = reinterpret_cast<fd::RowBlock*>(c->pool + o_rb);
    c->plan.cu_q = reinterpret_cast<int*>(c->pool + o_cuq);
    c->plan.cu_tiles = reinterpret_cast<int*>(c->pool + o_cut);
    c->plan.seq_bad = reinterpret_cast<int*>(c->pool + o_ok);
    c->plan.seg_count = reinterpret_cast<int*>(c->pool + o_sc);
    c->plan.cta_first = reinterpret_cast<int*>(c->pool + o_cf);
    c->plan.cta_start = reinterpret_cast<int*>(c->pool + o_cs);
    c->plan.cu_ne = reinterpret_cast<int*>(c->pool + o_cne);
    c->part.o = reinterpret_cast<float*>(c->pool + o_po);
    c->part.m = reinterpret_cast<float*>(c->pool + o_pm);
    c->part.l = reinterpret_cast<float*>(c->pool + o_pl);
    c->keys = reinterpret_cast<unsigned long long*>(c->pool + o_keys);
    c->ticket = reinterpret_cast<unsigned int*>(c->pool + o_tick);
    c->ds_key = reinterpret_cast<unsigned long long*>(c->pool + o_dsk);
    c->ds_sum = reinterpret_cast<float*>(c->pool + o_dss);
    c->ds_ticket = reinterpret_cast<unsigned int*>(c->pool + o_dst);
    c->ds_row_ticket = reinterpret_cast<unsigned int*>(c->pool + o_dsr);
    c->sv_part = reinterpret_cast<float2*>(c->pool + o_svp);
    c->sv_row = reinterpret_cast<float2*>(c->pool + o_svr);
    c->sv_row_ticket = reinterpret_cast<unsigned int*>(c->pool + o_svrt);
    c->sv_ticket = reinterpret_cast<unsigned int*>(c->pool + o_svt);
    c->sv_seq_ticket = reinterpret_cast<unsigned int*>(c->pool + o_svst);
    c->sv_seq = reinterpret_cast<int4*>(c->pool + o_svs);
    c->sv_chunk_w = reinterpret_cast<float*>(c->pool + o_svw);
    c->sv_flags = c->pool + o_svf;
    c->status = reinterpret_cast<int*>(c->pool + o_stat);
    *out = c;
    return FD_OK;
}

fd_status fd_destroy(fd_ctx* c) {
    if (!c) return FD_OK;
    cudaDeviceSynchronize();
    fd::attn_tc_free(c->tc_state);
    if (c->host) {
        HostStage* h = c->host;
        cudaStreamDestroy(h->h2d); cudaStreamDestroy(h->d2h);
        cudaEvent_t evs[] = {h->start, h->meta, h->logits, h->done, h->fin, h->q_ready[0], h->q_ready[1],
                             h->attn_done[0], h->attn_done[1], h->out_copied[0], h->out_copied[1]};
        for (cudaEvent_t e : evs) cudaEventDestroy(e);
        cudaFree(h->pool);
        delete h;
    }
    cudaFree(c->pool);
    delete c;
    return FD_OK;
}

fd_status fd_host_reserve(fd_ctx* c, int max_total_q_rows, int max_total_cand_rows) {
    if (!c || max_total_q_rows < 0 || max_total_cand_rows < 0) return FD_ERR_INVALID_ARG;
    if (c->host) return (max_total_q_rows <= c->host->max_q_rows && max_total_cand_rows <= c->host->max_cand_rows)
                            ? FD_OK : FD_ERR_INVALID_ARG;  // reserve once, with the maxima
    HostStage* h = new (std::nothrow) HostStage();
    if (!h) return FD_ERR_WORKSPACE;
    h->max_q_rows = max_total_q_rows; h->max_cand_rows = max_total_cand_rows;
    const int B = c->cfg.max_batch;
    const size_t qb = (size_t)max_total_q_rows * c->cfg.n_q_heads * c->cfg.head_dim * 2;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_q0 = take(qb), o_q1 = take(qb), o_o0 = take(qb), o_o1 = take(qb);
    const size_t kb = (size_t)max_total_q_rows * c->cfg.n_kv_heads * c->cfg.head_dim * 2;
    const size_t o_k0 = take(kb), o_k1 = take(kb), o_v0 = take(kb), o_v1 = take(kb);
    const size_t o_lg = take((size_t)max_total_cand_rows * c->cfg.vocab * 4);
    const size_t o_dr = take((size_t)max_total_cand_rows * 4);
    const size_t o_pt = take((size_t)B * c->cfg.max_pages_per_seq * 4);
    const size_t o_pl = take(B * 4), o_ql = take(B * 4), o_nm = take(B * 4), o_nb = take(B * 4), o_ac = take(B * 4), o_bo = take(B * 4);
    const size_t n_fr = (size_t)B * ((c->cfg.max_q_len + 15) / 16 + 1);
    const size_t o_fr = take(n_fr * 4), o_nf = take(4);
    if (cudaMalloc(&h->pool, off) != cudaSuccess) { cudaGetLastError(); delete h; return FD_ERR_WORKSPACE; }
    bool ok = cudaStreamCreateWithFlags(&h->h2d, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&h->d2h, cudaStreamNonBlocking) == cudaSuccess;
    cudaEvent_t* evs[] = {&h->start, &h->meta, &h->logits, &h->done, &h->fin, &h->q_ready[0], &h->q_ready[1],
                          &h->attn_done[0], &h->attn_done[1], &h->out_copied[0], &h->out_copied[1]};
    for (cudaEvent_t* e : evs) ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { cudaGetLastError(); cudaFree(h->pool); delete h; return FD_ERR_CUDA; }
    h->q[0] = h->pool + o_q0; h->q[1] = h->pool + o_q1; h->out[0] = h->pool + o_o0; h->out[1] = h->pool + o_o1;
    h->kn[0] = h->pool + o_k0; h->kn[1] = h->pool + o_k1; h->vn[0] = h->pool + o_v0; h->vn[1] = h->pool + o_v1;
    h->lg = reinterpret_cast<float*>(h->pool + o_lg);
    h->drafts = reinterpret_cast<int32_t*>(h->pool + o_dr); h->pt = reinterpret_cast<int32_t*>(h->pool + o_pt);
    h->pl = reinterpret_cast<int32_t*>(h->pool + o_pl); h->ql = reinterpret_cast<int32_t*>(h->pool + o_ql);
    h->nm = reinterpret_cast<int32_t*>(h->pool + o_nm); h->nb = reinterpret_cast<int32_t*>(h->pool + o_nb);
    h->acc = reinterpret_cast<int32_t*>(h->pool + o_ac);
    h->bon = reinterpret_cast<int32_t*>(h->pool + o_bo); h->freed = reinterpret_cast<int32_t*>(h->pool + o_fr);
    h->nfreed = reinterpret_cast<int32_t*>(h->pool + o_nf);
    c->host = h;
    return FD_OK;
}

fd_status fd_step_host(fd_ctx* c, int batch, int total_q_rows, int total_cand_rows, int n_layers,
                       const void* const* kv_caches, int num_pages, const void* q_host, void* out_host,
                       const float* logits_host, const int32_t* draft_tokens_host, int32_t* page_table_host,
                       int32_t* prefix_lens_host, const int32_t* q_lens_host, const int32_t* n_mask_host,
                       const int32_t* n_blocks_host, int32_t* accepted_len_host, int32_t* bonus_token_host, int32_t* freed_pages_host,
                       int32_t* n_freed_host, void* stream) {
    return fd_step_host_append(c, batch, total_q_rows, total_cand_rows, n_layers, const_cast<void* const*>(kv_caches), num_pages, q_host,
                               nullptr, nullptr, out_host, logits_host, draft_tokens_host, page_table_host, prefix_lens_host, q_lens_host,
                               n_mask_host, n_blocks_host, accepted_len_host, bonus_token_host, freed_pages_host, n_freed_host, stream);
}

fd_status fd_step_host_append(fd_ctx* c, int batch, int total_q_rows, int total_cand_rows, int n_layers,
                              void* const* kv_caches, int num_pages, const void* q_host, const void* k_new_host,
                              const void* v_new_host, void* out_host, const float* logits_host,
                              const int32_t* draft_tokens_host, int32_t* page_table_host, int32_t* prefix_lens_host,
                              const int32_t* q_lens_host, const int32_t* n_mask_host, const int32_t* n_blocks_host,
                              int32_t* accepted_len_host, int32_t* bonus_token_host, int32_t* freed_pages_host,
                              int32_t* n_freed_host, void* stream) {
    if (!c || !c->host) return FD_ERR_INVALID_ARG;
    if ((k_new_host == nullptr) != (v_new_host == nullptr)) return FD_ERR_INVALID_ARG;
    const bool append = k_new_host != nullptr;
    const size_t knb = (size_t)total_q_rows * c->cfg.n_kv_heads * c->cfg.head_dim * 2;
    HostStage* h = c->host;
    if (batch <= 0 || batch > c->cfg.max_batch || n_layers <= 0 || total_q_rows < 0 || total_cand_rows < 0 ||
        total_q_rows > h->max_q_rows || total_cand_rows > h->max_cand_rows)
        return FD_ERR_INVALID_ARG;
    if (!kv_caches || !q_host || !out_host || !page_table_host || !prefix_lens_host || !q_lens_host || !n_mask_host ||
        !accepted_len_host || !bonus_token_host || !freed_pages_host || !n_freed_host ||
        (total_cand_rows > 0 && (!logits_host || !draft_tokens_host)))
        return FD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // between the calls of this step the stream holds nothing but this library's launches and event waits
    struct BackToBack {
        fd_ctx* c; bool saved;
        explicit BackToBack(fd_ctx* c_) : c(c_), saved(c_->back_to_back) { c->back_to_back = true; }
        ~BackToBack() { c->back_to_back = saved; }
    } back_to_back(c);
    const size_t qb = (size_t)total_q_rows * c->cfg.n_q_heads * c->cfg.head_dim * 2;
    const size_t ptb = (size_t)batch * c->cfg.max_pages_per_seq * 4, lb = (size_t)batch * 4;
    const size_t n_fr = (size_t)batch * ((c->cfg.max_q_len + 15) / 16 + 1);
    bool ok = true;
    auto chk = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };
    const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;

    // everything of this step is ordered after what the caller already put on `stream`
    chk(cudaEventRecord(h->start, s));
    chk(cudaStreamWaitEvent(h->h2d, h->start, 0));
    chk(cudaStreamWaitEvent(h->d2h, h->start, 0));
    chk(cudaMemcpyAsync(h->pt, page_table_host, ptb, H2D, h->h2d));
    chk(cudaMemcpyAsync(h->pl, prefix_lens_host, lb, H2D, h->h2d));
    chk(cudaMemcpyAsync(h->ql, q_lens_host, lb, H2D, h->h2d));
    chk(cudaMemcpyAsync(h->nm, n_mask_host, lb, H2D, h->h2d));
    if (n_blocks_host) chk(cudaMemcpyAsync(h->nb, n_blocks_host, lb, H2D, h->h2d));
    chk(cudaEventRecord(h->meta, h->h2d));
    chk(cudaStreamWaitEvent(s, h->meta, 0));
    fd_status st = FD_OK;
    for (int l = 0; l < n_layers && ok && st == FD_OK; ++l) {
        const int b = l & 1;
        // q of layer l goes up while layer l-1 computes; the staging pair is reused every other layer
        if (l >= 2) chk(cudaStreamWaitEvent(h->h2d, h->attn_done[b], 0));
        chk(cudaMemcpyAsync(h->q[b], static_cast<const unsigned char*>(q_host) + (size_t)l * qb, qb, H2D, h->h2d));
        if (append) {  // the block's K/V of this layer ride with its q
            chk(cudaMemcpyAsync(h->kn[b], static_cast<const unsigned char*>(k_new_host) + (size_t)l * knb, knb, H2D, h->h2d));
            chk(cudaMemcpyAsync(h->vn[b], static_cast<const unsigned char*>(v_new_host) + (size_t)l * knb, knb, H2D, h->h2d));
        }
        chk(cudaEventRecord(h->q_ready[b], h->h2d));
        if (l >= 1 && total_cand_rows > 0) {
            // the logits go up in n_layers - 1 slices, one behind each later q block, so that no q block ever
            // queues behind a large copy; each slice hides under one layer's attention
            const size_t total = (size_t)total_cand_rows * c->cfg.vocab * 4;
            const size_t per = ((total + (size_t)(n_layers - 1) - 1) / (size_t)(n_layers - 1) + 255) / 256 * 256;
            const size_t lo = std::min(total, per * (size_t)(l - 1)), hi = std::min(total, per * (size_t)l);
            if (hi > lo)
                chk(cudaMemcpyAsync(reinterpret_cast<unsigned char*>(h->lg) + lo,
                                    reinterpret_cast<const unsigned char*>(logits_host) + lo, hi - lo, H2D, h->h2d));
            if (l == n_layers - 1) {
                chk(cudaMemcpyAsync(h->drafts, draft_tokens_host, (size_t)total_cand_rows * 4, H2D, h->h2d));
                chk(cudaEventRecord(h->logits, h->h2d));
            }
        }
        chk(cudaStreamWaitEvent(s, h->q_ready[b], 0));
        if (l >= 2) chk(cudaStreamWaitEvent(s, h->out_copied[b], 0));
        if (l == 0 && n_layers > 1)  // one work list for all layers of the step
            st = fd_plan_pin(c, batch, total_q_rows, h->pl, h->ql, h->nm, n_blocks_host ? h->nb : nullptr, s);
        if (st == FD_OK && append)
            st = fd_kv_append(c, batch, total_q_rows, h->kn[b], h->vn[b], kv_caches[l], num_pages, h->pt, h->pl, h->ql, s);
        if (st == FD_OK)
            st = fd_attn_draft_verify_blocks(c, batch, total_q_rows, h->q[b], kv_caches[l], num_pages, h->pt, h->pl, h->ql, h->nm,
                                             n_blocks_host ? h->nb : nullptr, h->out[b], s);
        // on an error the events of this layer are still recorded, so that nothing queued on the copy streams
        // waits for an event that never comes
        chk(cudaEventRecord(h->attn_done[b], s));
        chk(cudaStreamWaitEvent(h->d2h, h->attn_done[b], 0));
        chk(cudaMemcpyAsync(static_cast<unsigned char*>(out_host) + (size_t)l * qb, h->out[b], qb, D2H, h->d2h));
        chk(cudaEventRecord(h->out_copied[b], h->d2h));
    }
    c->pinned = false;  // the commit below changes the lengths
    // A failed call leaves the three streams consistent: whatever was queued on the copy streams is joined back
    // into `stream` before the error is returned, so no stream is left waiting and the staging may be reused.
    auto fail = [&](fd_status code) {
        cudaEventRecord(h->fin, h->h2d);
        cudaStreamWaitEvent(s, h->fin, 0);
        cudaEventRecord(h->done, h->d2h);
        cudaStreamWaitEvent(s, h->done, 0);
        cudaGetLastError();
        return code;
    };
    if (st != FD_OK) return fail(st);
    if (n_layers < 2 && total_cand_rows > 0) {
        chk(cudaMemcpyAsync(h->lg, logits_host, (size_t)total_cand_rows * c->cfg.vocab * 4, H2D, h->h2d));
        chk(cudaMemcpyAsync(h->drafts, draft_tokens_host, (size_t)total_cand_rows * 4, H2D, h->h2d));
        chk(cudaEventRecord(h->logits, h->h2d));
    }
    if (total_cand_rows > 0) chk(cudaStreamWaitEvent(s, h->logits, 0));
    st = fd_verify_accept(c, batch, total_cand_rows, h->lg, h->drafts, h->ql, h->nm, h->acc, h->bon, s);
    if (st != FD_OK) return fail(st);
    st = fd_kv_commit(c, batch, h->pt, h->pl, h->ql, h->acc, h->freed, h->nfreed, s);
    if (st != FD_OK) return fail(st);
    chk(cudaEventRecord(h->done, s));
    chk(cudaStreamWaitEvent(h->d2h, h->done, 0));
    chk(cudaMemcpyAsync(accepted_len_host, h->acc, lb, D2H, h->d2h));
    chk(cudaMemcpyAsync(bonus_token_host, h->bon, lb, D2H, h->d2h));
    chk(cudaMemcpyAsync(page_table_host, h->pt, ptb, D2H, h->d2h));
    chk(cudaMemcpyAsync(prefix_lens_host, h->pl, lb, D2H, h->d2h));
    chk(cudaMemcpyAsync(freed_pages_host, h->freed, n_fr * 4, D2H, h->d2h));
    chk(cudaMemcpyAsync(n_freed_host, h->nfreed, 4, D2H, h->d2h));
    chk(cudaEventRecord(h->fin, h->d2h));
    chk(cudaStreamWaitEvent(s, h->fin, 0));  // `stream` is complete only when every result is on the host
    if (!ok) return fail(FD_ERR_CUDA);
    return FD_OK;
}

int fd_attn_path(const fd_ctx* c) { return c ? c->attn_path : -1; }

int fd_attn_last_mode(const fd_ctx* c) { return c ? c->last_mode : -1; }

int64_t fd_launch_count(const fd_ctx* c) { return c ? c->launches : 0; }

fd_status fd_attn_draft_verify(fd_ctx* c, int batch, int total_q_rows, const void* q, const void* kv_cache,
                               int num_pages, const int32_t* page_table, const int32_t* prefix_lens,
                               const int32_t* q_lens, const int32_t* n_mask, void* out, void* stream) {
    return fd_attn_draft_verify_blocks(c, batch, total_q_rows, q, kv_cache, num_pages, page_table, prefix_lens, q_lens,
                                       n_mask, nullptr, out, stream);
}

fd_status fd_attn_draft_verify_blocks(fd_ctx* c, int batch, int total_q_rows, const void* q, const void* kv_cache,
                                      int num_pages, const int32_t* page_table, const int32_t* prefix_lens,
                                      const int32_t* q_lens, const int32_t* n_mask, const int32_t* n_blocks,
                                      void* out, void* stream) {
    if (!c || batch < 0 || total_q_rows < 0 || num_pages < 0) return FD_ERR_INVALID_ARG;
    if (batch > c->cfg.max_batch || (long long)total_q_rows > (long long)batch * c->cfg.max_q_len)
        return FD_ERR_INVALID_ARG;
    if (batch == 0) return total_q_rows == 0 ? FD_OK : FD_ERR_INVALID_ARG;
    if (!page_table || !prefix_lens || !q_lens || !n_mask) return FD_ERR_INVALID_ARG;
    if (total_q_rows > 0 && (!q || !out)) return FD_ERR_INVALID_ARG;
    if (!kv_cache || num_pages == 0) return FD_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(out, 16) || !aligned(kv_cache, 128) || !aligned(page_table, 4)) return FD_ERR_INVALID_ARG;
    if ((long long)num_pages * 2 * c->cfg.n_kv_heads * 16 > 0x7fffffffLL) return FD_ERR_UNSUPPORTED;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    fd::AttnParams p = attn_params(c, batch, total_q_rows, prefix_lens, q_lens, n_mask, n_blocks);
    p.num_pages = num_pages;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.kv = static_cast<const __nv_bfloat16*>(kv_cache);
    p.page_table = page_table;
    p.out = static_cast<__nv_bfloat16*>(out);

    const bool tc = c->attn_path == FD_ATTN_TCGEN05 && total_q_rows > 0;  // no rows: the plan alone checks the lengths
    if (tc) {
        if (fd::attn_tc_prepare(&c->tc_state, p) != cudaSuccess) { cudaGetLastError(); return FD_ERR_CUDA; }
    }
    c->epoch = c->epoch == 0x7fffffff ? 1 : c->epoch + 1;
    p.epoch = c->epoch;
    // a pinned plan serves this call if it was made for exactly these lengths; anything else replaces it
    const bool reuse = c->pinned && batch == c->pin_batch && total_q_rows == c->pin_rows && prefix_lens == c->pin_pl &&
                       q_lens == c->pin_ql && n_mask == c->pin_nm && n_blocks == c->pin_nb;
    // How the tensor-core kernel finds its work.  A call of few segments runs one cluster per segment; a call of
    // few sequences plans for itself (unless a pinned plan is there to use); everything else uses the plan kernel.
    int mode = fd::kTcPlanned;
    if (tc && p.rb_per_seq == 1 && c->tc_choice != FD_ATTN_TCGEN05_PLANNED) {
        const int n_seg = batch * p.Hkv;
        // (a table too narrow for four tiles per sequence leaves a cluster nothing to split)
        const bool splittable = (long long)p.max_pages * 16 >= 4 * fd::kTileTokens;
        const int cl = (c->tc_choice == FD_ATTN_TCGEN05 && batch <= fd::kSelfPlanMaxRb && n_seg <= fd::kClusterMaxSegments && splittable)
                           ? fd::attn_tc_cluster_size(c->tc_state, n_seg, c->n_sms) : 0;
        if (cl >= 2) { mode = fd::kTcCluster; p.cluster = cl; }
        else if (batch <= fd::kSelfPlanMaxRb && !reuse) mode = fd::kTcSelfPlanned;
    }
    if (mode == fd::kTcPlanned && !reuse) {
        c->pinned = false;
        fd::launch_plan(p, s);
        c->launches += 1;
    }
    // under a pinned plan, behind another call it served: the plan, the lengths and the page table are not what the
    // launch before this one writes, and may be read while it still runs
    p.early = (reuse && c->pinned && c->pin_chain) ? 1 : 0;
    if (!p.early) c->chain_out.clear();
    // ... and so may q and the cache, if no call of the chain writes them: the attention calls before this one write
    // their `out` (several of them may still be running: each starts as the one before it retires CTAs, and waits for
    // it only before its own first write), the append writes the cache
    if (p.early && tc && c->back_to_back) {
        const uintptr_t q0 = reinterpret_cast<uintptr_t>(q), q1 = q0 + (size_t)total_q_rows * p.Hq * p.d * 2;
        const uintptr_t k0 = reinterpret_cast<uintptr_t>(kv_cache), k1 = k0 + (size_t)num_pages * 2 * p.Hkv * 16 * p.d * 2;
        bool clash = c->chain_out.size() >= 1024;  // (a chain that long is not a step of a model: stop keeping track)
        for (const auto& w : c->chain_out) clash = clash || (w.first < q1 && q0 < w.second) || (w.first < k1 && k0 < w.second);
        // (behind the append, which writes the block's own slots of this cache: everything but those is read ahead)
        if (!clash) p.early = c->chain_append ? 3 : 2;
    }
    if (total_q_rows > 0 && c->chain_out.size() < 1024) {
        const uintptr_t o0 = reinterpret_cast<uintptr_t>(out);
        c->chain_out.emplace_back(o0, o0 + (size_t)total_q_rows * p.Hq * p.d * 2);
    }
    c->chain_append = false;
    c->after_attn = tc;
    c->pin_chain = reuse && c->pinned;
    if (c->attn_path == FD_ATTN_TCGEN05 && !tc) {
    } else if (tc) {
        fd::launch_attn_tc(c->tc_state, p, mode, s);  // merges split segments in its own epilogue
        c->launches += 1;
        c->last_mode = mode;
    } else {
        fd::launch_attn_simt(p, s);
        fd::launch_merge(p, s);
        c->launches += 2;
    }
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_plan_pin(fd_ctx* c, int batch, int total_q_rows, const int32_t* prefix_lens, const int32_t* q_lens,
                      const int32_t* n_mask, const int32_t* n_blocks, void* stream) {
    if (!c || batch <= 0 || total_q_rows < 0) return FD_ERR_INVALID_ARG;
    if (batch > c->cfg.max_batch || (long long)total_q_rows > (long long)batch * c->cfg.max_q_len) return FD_ERR_INVALID_ARG;
    if (!prefix_lens || !q_lens || !n_mask) return FD_ERR_INVALID_ARG;
    const fd::AttnParams p = attn_params(c, batch, total_q_rows, prefix_lens, q_lens, n_mask, n_blocks);
    fd::launch_plan(p, static_cast<cudaStream_t>(stream));
    c->launches += 1;
    c->pinned = true;
    c->pin_chain = false;  // the first call it serves comes right behind the plan kernel and waits for it
    c->after_attn = false;
    c->pin_batch = batch; c->pin_rows = total_q_rows;
    c->pin_pl = prefix_lens; c->pin_ql = q_lens; c->pin_nm = n_mask; c->pin_nb = n_blocks;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

namespace {
struct ScanAt {  // read access to a host scan, callable from the host-and-device range cutter
    const long long* a;
    __host__ __device__ long long operator()(int b) const { return a[b]; }
};
}  // namespace

fd_status fd_plan_ranges_host(int batch, int n_kv_heads, const int32_t* prefix_lens, const int32_t* q_lens, int n_ranges,
                              int32_t* range_start) {
    if (batch <= 0 || n_kv_heads <= 0 || n_ranges <= 0 || !prefix_lens || !q_lens || !range_start) return FD_ERR_INVALID_ARG;
    std::vector<long long> ct(batch + 1, 0), ne(batch + 1, 0);
    for (int b = 0; b < batch; ++b) {
        if (prefix_lens[b] < 0 || q_lens[b] < 0) return FD_ERR_INVALID_ARG;
        const long long t = q_lens[b] > 0 ? ((long long)prefix_lens[b] + q_lens[b] + fd::kTileTokens - 1) / fd::kTileTokens : 0;
        ct[b + 1] = ct[b] + t;
        ne[b + 1] = ne[b] + (t > 0);
    }
    const long long total = ct[batch] * n_kv_heads, k = FD_PIECE_COST;
    if (total > 0x7fffffffLL) return FD_ERR_UNSUPPORTED;
    const long long W = (long long)n_kv_heads * (ct[batch] + k * ne[batch]);
    const int n_use = fd::ranges_in_use(W, k, FD_MIN_RANGE_TILES, n_ranges);
    for (int c = 0; c <= n_ranges; ++c) {
        int first;
        range_start[c] = (c >= n_use || total == 0)
                             ? (int)total
                             : fd::range_cut(c, n_use, W, batch, n_kv_heads, k, ScanAt{ct.data()}, ScanAt{ne.data()}, &first);
    }
    return FD_OK;
}

fd_status fd_step_device(fd_ctx* c, int batch, int total_q_rows, int total_cand_rows, int n_layers, const void* const* q,
                         const void* const* k_new, const void* const* v_new, void* const* kv_caches, void* const* out,
                         int num_pages, int32_t* page_table, int32_t* prefix_lens, const int32_t* q_lens, const int32_t* n_mask,
                         const int32_t* n_blocks, const float* logits, const int32_t* draft_tokens, int32_t* accepted_len,
                         int32_t* bonus_token, int32_t* freed_pages, int32_t* n_freed, void* stream) {
    if (!c || n_layers <= 0 || !q || !kv_caches || !out || (k_new == nullptr) != (v_new == nullptr)) return FD_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l)
        if (!kv_caches[l] || (total_q_rows > 0 && (!q[l] || !out[l])) || (k_new && total_q_rows > 0 && (!k_new[l] || !v_new[l])))
            return FD_ERR_INVALID_ARG;
    // the stream holds nothing but this library's launches between the calls below
    struct BackToBack {
        fd_ctx* c; bool saved;
        explicit BackToBack(fd_ctx* c_) : c(c_), saved(c_->back_to_back) { c->back_to_back = true; }
        ~BackToBack() { c->back_to_back = saved; }
    } back_to_back(c);
    fd_status st = FD_OK;
    if (n_layers > 1) st = fd_plan_pin(c, batch, total_q_rows, prefix_lens, q_lens, n_mask, n_blocks, stream);  // one work list for all layers
    for (int l = 0; l < n_layers && st == FD_OK; ++l) {
        if (k_new && total_q_rows > 0)
            st = fd_kv_append(c, batch, total_q_rows, k_new[l], v_new[l], kv_caches[l], num_pages, page_table, prefix_lens, q_lens, stream);
        if (st == FD_OK)
            st = fd_attn_draft_verify_blocks(c, batch, total_q_rows, q[l], kv_caches[l], num_pages, page_table, prefix_lens, q_lens, n_mask,
                                             n_blocks, out[l], stream);
    }
    if (n_layers > 1) fd_plan_unpin(c);  // (no launch; the commit below would drop the pin anyway)
    if (st != FD_OK) return st;
    st = fd_verify_accept(c, batch, total_cand_rows, logits, draft_tokens, q_lens, n_mask, accepted_len, bonus_token, stream);
    if (st != FD_OK) return st;
    return fd_kv_commit(c, batch, page_table, prefix_lens, q_lens, accepted_len, freed_pages, n_freed, stream);
}

fd_status fd_calls_back_to_back(fd_ctx* c, int on) {
    if (!c) return FD_ERR_INVALID_ARG;
    c->back_to_back = on != 0;
    return FD_OK;
}

fd_status fd_plan_unpin(fd_ctx* c) {
    if (!c) return FD_ERR_INVALID_ARG;
    c->pinned = false;
    c->pin_chain = false;
    return FD_OK;
}

fd_status fd_verify_accept(fd_ctx* c, int batch, int total_cand_rows, const float* logits,
                           const int32_t* draft_tokens, const int32_t* q_lens, const int32_t* n_mask,
                           int32_t* accepted_len, int32_t* bonus_token, void* stream) {
    const bool after_attn = c && c->after_attn;  // (read before it is cleared: the sweep may be chained to that call)
    if (c) { c->pin_chain = false; c->after_attn = false; }  // (not an attention or append call)
    if (!c || batch < 0 || total_cand_rows < 0) return FD_ERR_INVALID_ARG;
    if (batch > c->cfg.max_batch || total_cand_rows > c->max_rows) return FD_ERR_INVALID_ARG;
    if (batch == 0) return total_cand_rows == 0 ? FD_OK : FD_ERR_INVALID_ARG;
    if (!q_lens || !n_mask || !accepted_len || !bonus_token) return FD_ERR_INVALID_ARG;
    if (total_cand_rows > 0 && (!logits || !draft_tokens)) return FD_ERR_INVALID_ARG;
    if (!aligned(logits, 4)) return FD_ERR_INVALID_ARG;
    const long long ctas = (long long)total_cand_rows * ((c->cfg.vocab + fd::kAcceptChunk - 1) / fd::kAcceptChunk);
    if (ctas > 0x7fffffffLL) return FD_ERR_UNSUPPORTED;
    fd::AcceptParams p;
    p.batch = batch; p.total_rows = total_cand_rows; p.vocab = c->cfg.vocab;
    p.logits = logits; p.drafts = draft_tokens; p.q_lens = q_lens; p.n_mask = n_mask;
    p.accepted = accepted_len; p.bonus = bonus_token;
    p.keys = c->keys; p.ticket = c->ticket; p.status = c->status;
    // Right behind an attention call (the last layer's) the sweep need not wait for it: it reads the logits and the
    // draft tokens, which that call does not write, into scratch of its own; only the scan, which writes the results,
    // waits.  (Behind anything else this is an ordinary launch.)
    p.chained = (after_attn && c->back_to_back) ? 1 : 0;
    fd::launch_accept(p, static_cast<cudaStream_t>(stream));
    c->launches += 1;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_verify_accept_sample(fd_ctx* c, int batch, int total_cand_rows, const float* logits, const float* draft_logits,
                                  const int32_t* draft_tokens, const int32_t* q_lens, const int32_t* n_mask, float temperature,
                                  const float* u_accept, const float* u_bonus, int32_t* accepted_len, int32_t* bonus_token,
                                  void* stream) {
    const bool after_attn = c && c->after_attn;  // (read before it is cleared: the sweep may be chained to that call)
    if (c) { c->pin_chain = false; c->after_attn = false; }  // (not an attention or append call)
    if (!c || batch < 0 || total_cand_rows < 0 || !(temperature > 0.f)) return FD_ERR_INVALID_ARG;
    if (batch > c->cfg.max_batch || total_cand_rows > c->max_rows) return FD_ERR_INVALID_ARG;
    if (batch == 0) return total_cand_rows == 0 ? FD_OK : FD_ERR_INVALID_ARG;
    if (!q_lens || !n_mask || !accepted_len || !bonus_token || !u_bonus) return FD_ERR_INVALID_ARG;
    if (total_cand_rows > 0 && (!logits || !draft_tokens || !u_accept)) return FD_ERR_INVALID_ARG;
    if (!aligned(logits, 4) || !aligned(draft_logits, 4)) return FD_ERR_INVALID_ARG;
    const long long chunks = (c->cfg.vocab + fd::kAcceptChunk - 1) / fd::kAcceptChunk;
    if ((long long)total_cand_rows * chunks > 0x7fffffffLL) return FD_ERR_UNSUPPORTED;
    fd::SampleParams p;
    p.batch = batch; p.total_rows = total_cand_rows; p.vocab = c->cfg.vocab;
    p.kt = 1.4426950408889634f / temperature;
    p.logits = logits; p.draft_logits = draft_logits; p.drafts = draft_tokens; p.q_lens = q_lens; p.n_mask = n_mask;
    p.u_accept = u_accept; p.u_bonus = u_bonus; p.accepted = accepted_len; p.bonus = bonus_token;
    p.part = c->sv_part; p.row_stat = c->sv_row; p.row_ticket = c->sv_row_ticket; p.ticket = c->sv_ticket;
    p.seq_info = c->sv_seq; p.chunk_w = c->sv_chunk_w; p.seq_ticket = c->sv_seq_ticket; p.flags = c->sv_flags;
    p.status = c->status;
    p.chained = (after_attn && c->back_to_back) ? 1 : 0;
    c->launches += fd::launch_accept_sample(p, static_cast<cudaStream_t>(stream));
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_kv_commit(fd_ctx* c, int batch, int32_t* page_table, int32_t* prefix_lens, const int32_t* q_lens,
                       const int32_t* accepted_len, int32_t* freed_pages, int32_t* n_freed, void* stream) {
    if (c) { c->pin_chain = false; c->after_attn = false; }  // (not an attention or append call)
    if (!c || batch < 0 || batch > c->cfg.max_batch || !n_freed) return FD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (batch == 0) return cudaMemsetAsync(n_freed, 0, sizeof(int32_t), s) == cudaSuccess ? FD_OK : FD_ERR_CUDA;
    if (!page_table || !prefix_lens || !q_lens || !accepted_len || !freed_pages) return FD_ERR_INVALID_ARG;
    fd::CommitParams p;
    p.batch = batch; p.max_pages = c->cfg.max_pages_per_seq; p.page_size = c->cfg.page_size;
    p.page_table = page_table; p.prefix_lens = prefix_lens; p.q_lens = q_lens; p.accepted = accepted_len;
    p.freed = freed_pages; p.n_freed = n_freed; p.status = c->status;
    c->pinned = false;  // the commit rewrites prefix_lens: a work list made for the old lengths must not be reused
    fd::launch_commit(p, s);
    c->launches += 1;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_kv_append(fd_ctx* c, int batch, int total_q_rows, const void* k_new, const void* v_new, void* kv_cache,
                       int num_pages, const int32_t* page_table, const int32_t* prefix_lens, const int32_t* q_lens,
                       void* stream) {
    if (!c || batch < 0 || batch > c->cfg.max_batch || total_q_rows < 0 || num_pages < 0) return FD_ERR_INVALID_ARG;
    if (batch == 0) return total_q_rows == 0 ? FD_OK : FD_ERR_INVALID_ARG;
    if (!page_table || !prefix_lens || !q_lens || !kv_cache) return FD_ERR_INVALID_ARG;
    if (total_q_rows > 0 && (!k_new || !v_new)) return FD_ERR_INVALID_ARG;
    if (!aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(kv_cache, 16)) return FD_ERR_INVALID_ARG;
    fd::AppendParams p;
    p.batch = batch; p.total_rows = total_q_rows; p.num_pages = num_pages; p.Hkv = c->cfg.n_kv_heads; p.d = c->cfg.head_dim;
    p.max_pages = c->cfg.max_pages_per_seq; p.max_q_len = c->cfg.max_q_len;
    p.k_new = static_cast<const __nv_bfloat16*>(k_new); p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.kv = static_cast<__nv_bfloat16*>(kv_cache);
    p.page_table = page_table; p.prefix_lens = prefix_lens; p.q_lens = q_lens; p.status = c->status;
    // Behind an attention call of a pinned chain the append need not wait for it: it reads the block's K/V, the page
    // table and the lengths, none of which the calls of the chain write (their `out` ranges are checked), and writes a
    // cache that only the NEXT attention call reads.  Its copies then run under that call's merge tail; it waits for the
    // call before it ends, so the attention call behind it, which waits for the append, has waited for both.
    p.chained = 0;
    if (c->back_to_back && c->pin_chain && c->pinned && !c->chain_append) {
        const size_t nb = (size_t)total_q_rows * p.Hkv * p.d * 2;
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(k_new), b0 = reinterpret_cast<uintptr_t>(v_new);
        bool clash = c->chain_out.size() >= 1024;
        for (const auto& w : c->chain_out) clash = clash || (w.first < a0 + nb && a0 < w.second) || (w.first < b0 + nb && b0 < w.second);
        p.chained = clash ? 0 : 1;
    }
    fd::launch_kv_append(p, static_cast<cudaStream_t>(stream));
    c->chain_append = true;  // the next attention call must not read the cache ahead of this launch
    c->after_attn = false;
    c->launches += 1;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_draft_select(fd_ctx* c, int batch, int total_mask_rows, int max_blocks, const float* draft_logits,
                          const float* bias, const int32_t* n_mask, const int32_t* n_blocks, float threshold,
                          int32_t* mask_tokens, float* mask_probs, int32_t* keep_len, void* stream) {
    const bool after_attn = c && c->after_attn;  // (read before it is cleared: the sweep may be chained to that call)
    if (c) { c->pin_chain = false; c->after_attn = false; }  // (not an attention or append call)
    if (!c || batch < 0 || batch > c->cfg.max_batch || total_mask_rows < 0 || total_mask_rows > c->max_rows || max_blocks < 1)
        return FD_ERR_INVALID_ARG;
    if (batch == 0) return total_mask_rows == 0 ? FD_OK : FD_ERR_INVALID_ARG;
    if (!n_mask || !keep_len || !(threshold >= 0.f)) return FD_ERR_INVALID_ARG;
    if (total_mask_rows > 0 && (!draft_logits || !mask_tokens || !mask_probs)) return FD_ERR_INVALID_ARG;
    const long long ctas = (long long)total_mask_rows * ((c->cfg.vocab + fd::kAcceptChunk - 1) / fd::kAcceptChunk);
    if (ctas > 0x7fffffffLL) return FD_ERR_UNSUPPORTED;
    fd::DraftSelectParams p;
    p.batch = batch; p.total_rows = total_mask_rows; p.vocab = c->cfg.vocab; p.max_blocks = max_blocks;
    p.logits = draft_logits; p.bias = bias; p.n_mask = n_mask; p.n_blocks = n_blocks; p.threshold = threshold;
    p.tokens = mask_tokens; p.probs = mask_probs; p.keep_len = keep_len;
    p.part_key = c->ds_key; p.part_sum = c->ds_sum; p.ticket = c->ds_ticket; p.row_ticket = c->ds_row_ticket; p.status = c->status;
    p.chained = (after_attn && c->back_to_back) ? 1 : 0;
    fd::launch_draft_select(p, static_cast<cudaStream_t>(stream));
    c->launches += 1;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_select_branch(fd_ctx* c, int batch, int max_block_len, const int32_t* mask_tokens, const int32_t* q_lens,
                           const int32_t* n_mask, const int32_t* n_blocks, const int32_t* accepted_len,
                           int32_t* next_draft, int32_t* next_len, void* stream) {
    if (c) { c->pin_chain = false; c->after_attn = false; }  // (not an attention or append call)
    if (!c || batch < 0 || batch > c->cfg.max_batch || max_block_len < 1) return FD_ERR_INVALID_ARG;
    if (batch == 0) return FD_OK;
    if (!q_lens || !n_mask || !accepted_len || !next_draft || !next_len) return FD_ERR_INVALID_ARG;
    fd::SelectParams p;
    p.batch = batch; p.max_kb = max_block_len; p.mask_tokens = mask_tokens; p.q_lens = q_lens; p.n_mask = n_mask;
    p.n_blocks = n_blocks; p.accepted = accepted_len; p.next_draft = next_draft; p.next_len = next_len;
    p.status = c->status;
    fd::launch_select_branch(p, static_cast<cudaStream_t>(stream));
    c->launches += 1;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_selftest_wait_timeout(fd_ctx* c, int limit_ms, void* stream) {
    if (c) { c->pin_chain = false; c->after_attn = false; }  // (not an attention or append call)
    if (!c || limit_ms < 1 || limit_ms > 1000) return FD_ERR_INVALID_ARG;
    fd::launch_wait_timeout_selftest(c->status, (unsigned long long)limit_ms * 1000000ull, static_cast<cudaStream_t>(stream));
    c->launches += 1;
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

fd_status fd_last_device_status(fd_ctx* c, int32_t* code, void* stream) {
    if (!c || !code) return FD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(code, c->status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return FD_ERR_CUDA;
    if (cudaMemsetAsync(c->status, 0, sizeof(int), s) != cudaSuccess) return FD_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FD_ERR_CUDA;
    if (*code & FD_DEV_TIMEOUT) {
        // a call that gave up may have left pieces counted on segments nobody merged: start the next call clean
        c->pinned = false;
        if (cudaMemsetAsync(c->plan.seg_count, 0, 2 * (size_t)c->max_rb * c->cfg.n_kv_heads * sizeof(int), s) != cudaSuccess) return FD_ERR_CUDA;
        // ... and a sweep that gave up leaves its running maxima and its row / call counters behind
        const size_t R = (size_t)c->max_rows, B = (size_t)c->cfg.max_batch;
        if (cudaMemsetAsync(c->keys, 0, R * sizeof(unsigned long long), s) != cudaSuccess ||
            cudaMemsetAsync(c->ticket, 0, sizeof(unsigned int), s) != cudaSuccess ||
            cudaMemsetAsync(c->ds_ticket, 0, sizeof(unsigned int), s) != cudaSuccess ||
            cudaMemsetAsync(c->ds_row_ticket, 0, R * sizeof(unsigned int), s) != cudaSuccess ||
            cudaMemsetAsync(c->sv_row_ticket, 0, R * sizeof(unsigned int), s) != cudaSuccess ||
            cudaMemsetAsync(c->sv_ticket, 0, sizeof(unsigned int), s) != cudaSuccess ||
            cudaMemsetAsync(c->sv_seq_ticket, 0, B * sizeof(unsigned int), s) != cudaSuccess)
            return FD_ERR_CUDA;
    }
    return FD_OK;
}

}  // extern "C"
