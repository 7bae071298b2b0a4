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
 *   - fdo_accept_stochastic: the same rule at temperature > 0, i.e. speculative
 *     sampling as Sec. 3 states it (accept by the ratio of target and drafter
 *     probabilities, bonus from the residual distribution).
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
    const int32_t *n_blocks;  /* [B] or NULL: mask blocks per sequence (0 / 1 / NULL = one block) */
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

/* Hybrid mask (Sec. 4.1; Fig. 2 caption; Eq. 2 for several blocks).  i = query row inside the
 * block, j = logical key position.  n = prefix length, C = candidate rows, M = mask rows, nb = mask
 * blocks.  The M mask tokens form nb consecutive blocks of M / nb tokens; block g is the next-draft
 * branch under the hypothesis that r = C - nb + g drafts are accepted (Eq. 2: conditioned on the
 * prefix and the first r drafts), so it sees the candidates 0..r -- row 0 being the known bonus
 * token -- and its own block in both directions; blocks never see each other, and clean rows never
 * see a mask token.  nb = 1 is the single block that sees every candidate. */
static int allowed(int i, int j, int n, int C, int M, int nb)
{
    if (j < n) return 1;                    /* everyone sees the clean prefix */
    int t = j - n;                          /* index of the key inside the query block */
    if (i < C) return t <= i;               /* clean row: causal, never sees a mask token */
    if (nb < 1) nb = 1;
    int kb = M / nb;                        /* tokens per mask block */
    int g = (i - C) / kb;                   /* block of this mask row */
    int r = C - nb + g;                     /* hypothesis: candidates 0..r are the verified context */
    if (t < C) return t <= r;               /* a candidate key */
    return (t - C) / kb == g;               /* a mask key: own block only */
}

/* one output row out[d] for sequence b, block row i, q-head h; row0 = first q row of b */
static void attn_row(const fdo_problem *p, int b, int64_t row0, int i, int h, double *out, double *w)
{
    const int d = p->d;
    const int n = p->prefix_lens[b], Lq = p->q_lens[b], M = p->n_mask[b], C = Lq - M;
    const int kv_len = n + Lq;
    const int nb = p->n_blocks ? p->n_blocks[b] : 1;
    const int g = h / (p->Hq / p->Hkv);
    const uint16_t *qv = p->q + ((row0 + i) * p->Hq + h) * (int64_t)d;

    double mx = -INFINITY;
    for (int j = 0; j < kv_len; ++j) {
        if (!allowed(i, j, n, C, M, nb)) { w[j] = -INFINITY; continue; }
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
    fdo_problem p = { Hq, Hkv, d, page_size, max_pages, NULL, q, kv, page_table,
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

/* Same with several mask blocks per sequence (the all-hypotheses form of parallel drafting, Eq. 2). */
void fdo_attn_blocks(int B, int Hq, int Hkv, int d, int page_size, int max_pages,
        const uint16_t *q, const uint16_t *kv, const int32_t *page_table,
        const int32_t *prefix_lens, const int32_t *q_lens, const int32_t *n_mask, const int32_t *n_blocks,
        double scale, double *out)
{
    fdo_problem p = make_problem(Hq, Hkv, d, page_size, max_pages, q, kv, page_table,
                                 prefix_lens, q_lens, n_mask, scale);
    p.n_blocks = n_blocks;
    int64_t row0 = 0;
    int max_kv = 1;
    for (int b = 0; b < B; ++b)
        if (prefix_lens[b] + q_lens[b] > max_kv) max_kv = prefix_lens[b] + q_lens[b];
    for (int b = 0; b < B; ++b) {
        const int Lq = q_lens[b];
        #pragma omp parallel
        {
            double *w = (double *)malloc(sizeof(double) * (size_t)max_kv);
            #pragma omp for collapse(2) schedule(dynamic)
            for (int i = 0; i < Lq; ++i)
                for (int h = 0; h < Hq; ++h)
                    attn_row(&p, b, row0, i, h, out + ((row0 + i) * Hq + h) * (int64_t)d, w);
            free(w);
        }
        row0 += Lq;
    }
}

/* Branch selection (Sec. 3, "Parallel speculative decoding": once verification has fixed r_acc, the
 * branch prepared under that hypothesis becomes the next draft).  mask_tokens [sum_b M_b] holds one
 * proposed token per mask row, sequence-major.  For sequence b with nb blocks of kb tokens the block
 * of hypothesis r is g = r - (C_b - nb); next_draft [B, max_kb] receives its kb tokens (padded with -1)
 * and next_len[b] = kb, or next_len[b] = 0 when that hypothesis was not prepared (g < 0), when the
 * sequence has no mask rows, or when accepted_len[b] < 0. */
void fdo_select_branch(int B, int max_kb, const int32_t *mask_tokens, const int32_t *q_lens, const int32_t *n_mask,
        const int32_t *n_blocks, const int32_t *accepted_len, int32_t *next_draft, int32_t *next_len)
{
    int64_t m0 = 0;
    for (int b = 0; b < B; ++b) {
        const int M = n_mask[b], C = q_lens[b] - M;
        int nb = n_blocks ? n_blocks[b] : 1;
        if (nb < 1) nb = 1;
        for (int u = 0; u < max_kb; ++u) next_draft[(int64_t)b * max_kb + u] = -1;
        next_len[b] = 0;
        if (M > 0 && accepted_len[b] >= 0) {
            const int kb = M / nb, g = accepted_len[b] - (C - nb);
            if (g >= 0 && g < nb) {
                for (int u = 0; u < kb; ++u) next_draft[(int64_t)b * max_kb + u] = mask_tokens[m0 + (int64_t)g * kb + u];
                next_len[b] = kb;
            }
        }
        m0 += M;
    }
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

/* Verification by speculative sampling (Sec. 3).  Each draft is kept or dropped by comparing the target
 * distribution p with the drafter distribution q at the drafted token; where the first draft is dropped, a
 * replacement is drawn from what is left of p once q has been taken out; committed length = accepted + 1.
 * The rule itself is the published speculative-sampling algorithm that Sec. 3 refers to.  Rows and
 * draft_tokens as in fdo_accept.
 *
 *   p_j = softmax(logits[r0 + j] / T)              target distribution after candidate row j
 *   q_j = softmax(draft_logits[r0 + j] / T)        distribution draft j + 1 was proposed from, or, with
 *                                                  draft_logits == NULL, all mass on the proposed token
 *   for j = 0 .. k-1, x = draft_tokens[r0 + j + 1]:
 *       accept x  iff  u_accept[r0 + j] * q_j(x) < p_j(x)      (for q_j(x) > 0 this is u < min(1, p/q), since
 *                                                  u < 1; written as a product it is also defined for a token
 *                                                  the drafter gives no mass: accepted iff p_j(x) > 0; a token
 *                                                  with p = q = 0 is rejected);  the first rejection ends the loop
 *   rejected at j:   bonus ~ max(0, p_j - q_j) normalised      all k accepted:   bonus ~ p_k
 *
 * Random numbers are inputs: u_accept [R] (the entry of a sequence's last row is unused) and u_bonus [B], all
 * in [0, 1).  A token is drawn from weights w by inverting the cumulative sum in index order: the first y
 * with w[0] + .. + w[y] > u * sum(w).  ratio [R] (optional) receives p_j(x) / q_j(x) for every tested draft
 * (-1 elsewhere; +inf or NaN where q_j(x) = 0) and weights [B, V] (optional) the unnormalised weights the
 * bonus token was drawn from, so that a test can tell a wrong decision from one that sits on a rounding
 * boundary. */
void fdo_accept_stochastic(int B, int V, const float *logits, const float *draft_logits, const int32_t *draft_tokens,
        const int32_t *q_lens, const int32_t *n_mask, double temperature, const float *u_accept,
        const float *u_bonus, int32_t *accepted_len, int32_t *bonus_token, double *ratio, double *weights)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    int64_t r0 = 0;
    for (int b = 0; b < B; ++b) {
        const int C = q_lens[b] - n_mask[b];
        if (C <= 0) { accepted_len[b] = -1; bonus_token[b] = -1; continue; }
        const int k = C - 1;
        int a = 0, rejected = 0;
        for (int j = 0; j <= k; ++j) {
            /* p_j, and q_j where there is a draft to test */
            const float *row = logits + (r0 + j) * (int64_t)V;
            double mx = row[0];
            for (int v = 1; v < V; ++v) if (row[v] > mx) mx = row[v];
            double z = 0.0;
            for (int v = 0; v < V; ++v) { p[v] = exp(((double)row[v] - mx) / temperature); z += p[v]; }
            for (int v = 0; v < V; ++v) p[v] /= z;
            if (ratio) ratio[r0 + j] = -1.0;
            if (j == k) break;               /* every draft accepted: the bonus comes from p_k */
            const int x = draft_tokens[r0 + j + 1];
            if (draft_logits) {
                const float *dr = draft_logits + (r0 + j) * (int64_t)V;
                double dm = dr[0];
                for (int v = 1; v < V; ++v) if (dr[v] > dm) dm = dr[v];
                double dz = 0.0;
                for (int v = 0; v < V; ++v) { q[v] = exp(((double)dr[v] - dm) / temperature); dz += q[v]; }
                for (int v = 0; v < V; ++v) q[v] /= dz;
            } else {
                for (int v = 0; v < V; ++v) q[v] = 0.0;
                q[x] = 1.0;
            }
            const double rho = p[x] / q[x];
            if (ratio) ratio[r0 + j] = rho;
            if ((double)u_accept[r0 + j] * q[x] < p[x]) { ++a; continue; }
            rejected = 1;
            for (int v = 0; v < V; ++v) { const double w = p[v] - q[v]; p[v] = w > 0.0 ? w : 0.0; }
            break;
        }
        (void)rejected;
        /* p now holds the weights of the bonus token: the residual, or p_k */
        double total = 0.0;
        for (int v = 0; v < V; ++v) total += p[v];
        const double target = (double)u_bonus[b] * total;
        double cum = 0.0;
        int tok = V - 1;
        for (int v = 0; v < V; ++v) { cum += p[v]; if (cum > target) { tok = v; break; } }
        accepted_len[b] = a;
        bonus_token[b] = tok;
        if (weights) memcpy(weights + (int64_t)b * V, p, sizeof(double) * (size_t)V);
        r0 += C;
    }
    free(p);
    free(q);
}

/* Draft-side tail of the step (Sec. 4.2, Eq. 4; Sec. 4.3 "Selective verification", Eq. 5).  One row of
 * draft logits per mask token, sequence-major.  With the calibration bias already evaluated by the caller
 * (the two-layer MLP of Eq. 4 needs trained weights), the calibrated logits are l~ = l + bias, the drafted
 * token of a row is argmax l~ (lowest index on ties) and its confidence p = softmax(l~)[token].  Within each
 * next-draft block (the M_b mask rows of a sequence are nb_b equal blocks) the cumulative confidence of
 * position i is the product of p over positions 1..i (Eq. 5: the estimate of P(L_acc >= i)); keep_len of
 * the block is the number of leading positions whose cumulative confidence is still >= threshold, i.e. how
 * many of its drafts are worth verifying in the next step.
 *
 * Eq. 4 defines the sum, not a precision: everything here is float64 (the float32 inputs convert exactly).
 * tokens [Rm], probs [Rm], cum [Rm], keep_len [B, max_blocks] (zero where a sequence has fewer blocks).
 * gap [Rm] (optional) receives the margin by which the winning calibrated logit beats the best other one
 * (0 on an exact tie, +inf when V = 1), so that a test can tell a wrong argmax from one that a
 * lower-precision sum may legitimately decide the other way. */
void fdo_draft_select(int B, int V, int max_blocks, const float *logits, const float *bias, const int32_t *n_mask,
        const int32_t *n_blocks, double threshold, int32_t *tokens, double *probs, double *cum, int32_t *keep_len,
        double *gap)
{
    int64_t r0 = 0;
    for (int b = 0; b < B; ++b) {
        const int M = n_mask[b];
        int nb = n_blocks ? n_blocks[b] : 1;
        if (nb < 1) nb = 1;
        for (int g = 0; g < max_blocks; ++g) keep_len[(int64_t)b * max_blocks + g] = 0;
        if (M <= 0) continue;
        const int kb = M / nb;
        for (int u = 0; u < M; ++u) {
            const float *lr = logits + (r0 + u) * (int64_t)V;
            const float *br = bias ? bias + (r0 + u) * (int64_t)V : NULL;
            int best = 0;
            double bestv = br ? (double)lr[0] + (double)br[0] : (double)lr[0];
            for (int v = 1; v < V; ++v) {
                const double x = br ? (double)lr[v] + (double)br[v] : (double)lr[v];
                if (x > bestv) { bestv = x; best = v; }
            }
            double den = 0.0, second = -INFINITY;
            for (int v = 0; v < V; ++v) {
                const double x = br ? (double)lr[v] + (double)br[v] : (double)lr[v];
                den += exp(x - bestv);
                if (v != best && x > second) second = x;
            }
            tokens[r0 + u] = best;
            probs[r0 + u] = 1.0 / den;
            if (gap) gap[r0 + u] = bestv - second;
        }
        for (int g = 0; g < nb; ++g) {
            double c = 1.0;
            int keep = 0, open = 1;
            for (int u = 0; u < kb; ++u) {
                c *= probs[r0 + (int64_t)g * kb + u];
                cum[r0 + (int64_t)g * kb + u] = c;
                if (open && c >= threshold) ++keep; else open = 0;
            }
            if (g < max_blocks) keep_len[(int64_t)b * max_blocks + g] = keep;
        }
        r0 += M;
    }
}

/* KV append ("append, then attend"): the K/V of the Lq_b query tokens of sequence b (candidates first, then
 * mask tokens) are written at logical positions n_b .. n_b + Lq_b - 1 of its paged cache, so that the
 * attention of this step, and after the commit every later step, finds them there (Sec. 4.1 "Inference": the
 * KV cache built by the target's own forward pass is what later steps reuse).  k_new, v_new [T, Hkv, d] bf16
 * bits, sequence-major rows; every other byte of the cache is left as it was. */
void fdo_kv_append(int B, int Hkv, int d, int page_size, int max_pages, const uint16_t *k_new, const uint16_t *v_new,
        uint16_t *kv, const int32_t *page_table, const int32_t *prefix_lens, const int32_t *q_lens)
{
    int64_t row = 0;
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < q_lens[b]; ++i, ++row) {
            const int j = prefix_lens[b] + i;
            const int64_t page = page_table[(int64_t)b * max_pages + j / page_size];
            const int slot = j % page_size;
            for (int h = 0; h < Hkv; ++h)
                for (int c = 0; c < d; ++c) {
                    kv[((((page * 2 + 0) * Hkv + h) * page_size + slot) * (int64_t)d) + c] = k_new[(row * Hkv + h) * (int64_t)d + c];
                    kv[((((page * 2 + 1) * Hkv + h) * page_size + slot) * (int64_t)d) + c] = v_new[(row * Hkv + h) * (int64_t)d + c];
                }
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
