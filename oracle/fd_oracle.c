/*
 * CPU oracle for the FlexDraft decode-step hot path.  TEST INFRASTRUCTURE ONLY:
 * nothing in the product path may link, import or call this file.  It shares no
 * code with the CUDA kernels.
 *
 * Everything is the plain definition, in float64, with no tiling, no online
 * softmax and no reordering:
 *
 *   - fdo_attn_row / fdo_attn: attention of one target forward pass whose query
 *     block per sequence is [bonus, k drafts, n_mask mask tokens] (paper Sec. 4.1,
 *     "Inference"), read against a paged KV cache under the hybrid mask of
 *     Sec. 4.1 / Fig. 2 caption: candidate (clean) rows are causal over the
 *     prefix and the earlier candidates ("identical to a standard forward pass");
 *     mask rows see the clean prefix, the candidates and their own block
 *     bidirectionally; clean rows never see a mask token.
 *   - fdo_accept: greedy (temperature 0) reading of the verification rule of
 *     Sec. 3: a draft is accepted while it equals the target argmax, the token at
 *     the first mismatch is the bonus token, committed length = accepted + 1.
 *   - fdo_commit: KV commit / rollback.  The paper only implies it (the clean KV
 *     cache "can be reused across all decoding steps", mask tokens are invisible
 *     to clean tokens); the reading implemented is: keep bonus + accepted drafts,
 *     drop everything after, release the pages no longer covered.
 *
 * Pins (tests/test_oracle_*.py): textbook causal decode attention, dense-mask
 * library attention on tiny inputs, softmax rows summing to one, mask invariance
 * properties, planted argmax positions, closed-form accept-length statistics,
 * page-accounting invariants, a greedy-decode replay.  The paper prints no worked
 * numeric example for this path, so parity with the authors' own implementation
 * is unpinned beyond those.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

typedef struct {
    int Hq, Hkv, d, page_size, max_pages;
    const uint16_t *q;        /* [T, Hq, d] bf16 bits */
    const uint16_t *kv;       /* [num_pages, 2, Hkv, page_size, d] bf16 bits */
    const int32_t *page_table;/* [B, max_pages] */
    const int32_t *prefix_lens, *q_lens, *n_mask;
    double scale;
} fdo_problem;

/* address of K (which=0) or V (which=1) of logical token j of sequence b, kv-head g */
static const uint16_t *kv_ptr(const fdo_problem *p, int b, int j, int which, int g)
{
    int64_t page = p->page_table[(int64_t)b * p->max_pages + j / p->page_size];
    int64_t slot = j % p->page_size;
    return p->kv + ((((page * 2 + which) * p->Hkv + g) * p->page_size + slot) * (int64_t)p->d);
}

/* Hybrid mask (Sec. 4.1; Fig. 2 caption).  i = query row inside the block,
 * j = logical key position.  n = prefix length, C = candidate rows, M = mask rows. */
static int allowed(int i, int j, int n, int C, int M)
{
    if (j < n) return 1;                    /* everyone sees the clean prefix */
    int t = j - n;                          /* index of the key inside the query block */
    if (i < C) return t <= i;               /* clean row: causal, never sees a mask token */
    (void)M;
    return 1;                               /* mask row: candidates + whole own block */
}

/* one output row out[d] for sequence b, block row i, q-head h; row0 = first q row of b */
static void attn_row(const fdo_problem *p, int b, int64_t row0, int i, int h, double *out, double *w)
{
    const int d = p->d;
    const int n = p->prefix_lens[b], Lq = p->q_lens[b], M = p->n_mask[b], C = Lq - M;
    const int kv_len = n + Lq;
    const int g = h / (p->Hq / p->Hkv);
    const uint16_t *qv = p->q + ((row0 + i) * p->Hq + h) * (int64_t)d;

    double mx = -INFINITY;
    for (int j = 0; j < kv_len; ++j) {
        if (!allowed(i, j, n, C, M)) { w[j] = -INFINITY; continue; }
        const uint16_t *kp = kv_ptr(p, b, j, 0, g);
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += bf16_to_f64(qv[c]) * bf16_to_f64(kp[c]);
        w[j] = s * p->scale;
        if (w[j] > mx) mx = w[j];
    }
    double den = 0.0;
    for (int j = 0; j < kv_len; ++j) {
        w[j] = (w[j] == -INFINITY) ? 0.0 : exp(w[j] - mx);
        den += w[j];
    }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = 0; j < kv_len; ++j) {
        if (w[j] == 0.0) continue;
        const uint16_t *vp = kv_ptr(p, b, j, 1, g);
        double pj = w[j] / den;
        for (int c = 0; c < d; ++c) out[c] += pj * bf16_to_f64(vp[c]);
    }
}

static fdo_problem make_problem(int Hq, int Hkv, int d, int page_size, int max_pages,
        const uint16_t *q, const uint16_t *kv, const int32_t *page_table,
        const int32_t *prefix_lens, const int32_t *q_lens, const int32_t *n_mask, double scale)
{
    fdo_problem p = { Hq, Hkv, d, page_size, max_pages, q, kv, page_table,
                      prefix_lens, q_lens, n_mask, scale };
    return p;
}

int fdo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Full attention: out [T, Hq, d] float64. */
void fdo_attn(int B, int Hq, int Hkv, int d, int page_size, int max_pages,
        const uint16_t *q, const uint16_t *kv, const int32_t *page_table,
        const int32_t *prefix_lens, const int32_t *q_lens, const int32_t *n_mask,
        double scale, double *out)
{
    fdo_problem p = make_problem(Hq, Hkv, d, page_size, max_pages, q, kv, page_table,
                                 prefix_lens, q_lens, n_mask, scale);
    int64_t *row0 = (int64_t *)malloc(sizeof(int64_t) * (size_t)(B + 1));
    int max_kv = 1;
    row0[0] = 0;
    for (int b = 0; b < B; ++b) {
        row0[b + 1] = row0[b] + q_lens[b];
        if (prefix_lens[b] + q_lens[b] > max_kv) max_kv = prefix_lens[b] + q_lens[b];
    }
    for (int b = 0; b < B; ++b) {
        const int Lq = q_lens[b];
        #pragma omp parallel
        {
            double *w = (double *)malloc(sizeof(double) * (size_t)max_kv);
            #pragma omp for collapse(2) schedule(dynamic)
            for (int i = 0; i < Lq; ++i)
                for (int h = 0; h < Hq; ++h)
                    attn_row(&p, b, row0[b], i, h, out + ((row0[b] + i) * Hq + h) * (int64_t)d, w);
            free(w);
        }
    }
    free(row0);
}

/* A single output row (sampled checks at sizes where the full pass is too slow). */
void fdo_attn_row(int Hq, int Hkv, int d, int page_size, int max_pages,
        const uint16_t *q, const uint16_t *kv, const int32_t *page_table,
        const int32_t *prefix_lens, const int32_t *q_lens, const int32_t *n_mask,
        double scale, int b, int i, int h, double *out_row)
{
    fdo_problem p = make_problem(Hq, Hkv, d, page_size, max_pages, q, kv, page_table,
                                 prefix_lens, q_lens, n_mask, scale);
    int64_t row0 = 0;
    for (int s = 0; s < b; ++s) row0 += q_lens[s];
    double *w = (double *)malloc(sizeof(double) * (size_t)(prefix_lens[b] + q_lens[b] + 1));
    attn_row(&p, b, row0, i, h, out_row, w);
    free(w);
}

/* Greedy verification (Sec. 3).  logits [R, V] holds candidate rows only, sequence
 * major; draft_tokens[r] is the token that was fed at candidate row r (row 0 of a
 * sequence = the previous bonus token, rows 1..k = the drafts).  argmax_out [R] is
 * optional.  Ties go to the lowest index.  A sequence without candidate rows gets
 * accepted_len = bonus = -1. */
void fdo_accept(int B, int V, const float *logits, const int32_t *draft_tokens,
        const int32_t *q_lens, const int32_t *n_mask,
        int32_t *accepted_len, int32_t *bonus_token, int32_t *argmax_out)
{
    int64_t r0 = 0;
    for (int b = 0; b < B; ++b) {
        const int C = q_lens[b] - n_mask[b];
        if (C <= 0) { accepted_len[b] = -1; bonus_token[b] = -1; continue; }
        const int k = C - 1;                 /* number of drafts under verification */
        int32_t *am = (int32_t *)malloc(sizeof(int32_t) * (size_t)C);
        for (int j = 0; j < C; ++j) {        /* target argmax of every candidate row */
            const float *row = logits + (r0 + j) * (int64_t)V;
            int best = 0;
            for (int v = 1; v < V; ++v)
                if (row[v] > row[best]) best = v;
            am[j] = best;
            if (argmax_out) argmax_out[r0 + j] = best;
        }
        int a = 0;                           /* r_acc: drafts accepted so far */
        while (a < k && am[a] == draft_tokens[r0 + a + 1]) ++a;
        accepted_len[b] = a;
        bonus_token[b] = am[a];              /* token at the first mismatch (or after the last draft) */
        free(am);
        r0 += C;
    }
}

/* KV commit / rollback.  In place on page_table [B, max_pages] and prefix_lens [B].
 * Sequences with accepted_len < 0 are left unchanged.  freed_pages is packed in
 * (sequence ascending, logical page ascending) order; returns the number freed. */
int fdo_commit(int B, int page_size, int max_pages, int32_t *page_table, int32_t *prefix_lens,
        const int32_t *q_lens, const int32_t *accepted_len, int32_t *freed_pages)
{
    int n_freed = 0;
    for (int b = 0; b < B; ++b) {
        if (accepted_len[b] < 0) continue;
        const int n = prefix_lens[b];
        const int new_len = n + accepted_len[b] + 1;
        const int old_pages = (n + q_lens[b] + page_size - 1) / page_size;
        const int keep = (new_len + page_size - 1) / page_size;
        for (int pg = keep; pg < old_pages; ++pg) {
            int32_t *e = page_table + (int64_t)b * max_pages + pg;
            freed_pages[n_freed++] = *e;
            *e = -1;
        }
        prefix_lens[b] = new_len;
    }
    return n_freed;
}
