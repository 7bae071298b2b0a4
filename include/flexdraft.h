/*
 * flexdraft.h -- C ABI of the FlexDraft decode-step hot path for NVIDIA B200 (sm_100a).
 *
 * One decode step of FlexDraft's parallel draft-and-verify decoding (paper Sec. 4.1,
 * "Inference"; Sec. 3 for the verification rule) is, per attention layer and per
 * sequence b, the attention of a query block
 *
 *        [ bonus token | k_b draft tokens | M_b mask tokens ]
 *          \____ C_b = k_b + 1 candidate rows ____/
 *
 * against that sequence's paged KV cache under the hybrid mask, followed, once per
 * step, by lossless verification of the drafts and by the commit / rollback of the KV
 * positions written for this block.  This library exports those three operations
 * (fd_attn_draft_verify, fd_verify_accept, fd_kv_commit) and the steps next to them: the
 * all-hypotheses form of the attention and the branch selection (Eq. 2), the draft-side
 * tail (Eq. 4, Eq. 5), verification by sampling at temperature > 0 (Sec. 3), the KV
 * append, and a whole step from host buffers.  Everything runs in hand-written CUDA
 * kernels; there is no CPU fallback.
 *
 * Conventions (all entry points)
 *   - "device pointer": memory on the GPU that is current when fd_create() ran, owned
 *     by the caller.  "host pointer": ordinary host memory, owned by the caller.
 *   - Calls are asynchronous on the given CUDA stream (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream) and ordered by it.  Calls that share one fd_ctx
 *     must be issued on one stream, or be ordered by the caller: they share the context's
 *     scratch memory.
 *     A context is not thread-safe: one host thread at a time per fd_ctx.
 *   - The hot calls (fd_attn_draft_verify, fd_verify_accept, fd_kv_commit) never allocate
 *     and never synchronise; all scratch memory is sized by fd_create() from fd_config.
 *   - Errors the host can see (NULL pointer, size beyond the configured maximum,
 *     unsupported shape, misaligned pointer) return a code and launch nothing.
 *   - Errors only the device can see (lengths that contradict each other, a page id
 *     outside the pool, ...) never trap: the kernels skip the work, write a defined
 *     value (documented per call) and OR a FD_DEV_* bit into a sticky status word that
 *     fd_last_device_status() reads.
 *
 * Notation: B sequences; Hq q-heads, Hkv kv-heads, G = Hq/Hkv; d = head_dim; P = page_size
 * (16 tokens); V = vocab.  n_b = prefix_lens[b]; Lq_b = q_lens[b]; M_b = n_mask[b];
 * C_b = Lq_b - M_b; kv_len_b = n_b + Lq_b; T = sum_b Lq_b; R = sum_b C_b.
 */
#ifndef FLEXDRAFT_H
#define FLEXDRAFT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fd_ctx fd_ctx; /* opaque; owns scratch memory and the device status word */

typedef enum {
    FD_OK = 0,
    FD_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, size beyond fd_config maximum */
    FD_ERR_UNSUPPORTED = 2,   /* shape outside what the kernels implement */
    FD_ERR_WORKSPACE = 3,     /* scratch memory could not be allocated */
    FD_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed */
    FD_ERR_DEVICE_STATUS = 5, /* reserved */
    FD_ERR_STATIC_LIMIT = 6   /* fd_verify_accept_static: more rows or sequences than its fixed scratch holds */
} fd_status;

/* Bits of the sticky device status word. */
enum {
    FD_DEV_BAD_LENGTHS = 1,   /* lengths negative, n_mask > q_len, q_len > max_q_len, kv_len beyond the
                                 page table, or row totals that do not match the call's row count */
    FD_DEV_BAD_PAGE = 2,      /* a page id needed by a sequence is outside [0, num_pages) */
    FD_DEV_TIMEOUT = 4,       /* a bounded device-side wait ran out; the kernel returned early */
    FD_DEV_BAD_ACCEPT = 8     /* fd_kv_commit: accepted_len[b] >= q_lens[b] */
};

/* Which attention kernel fd_attn_draft_verify launches. */
enum {
    FD_ATTN_AUTO = 0,         /* tensor-core kernel when the shape allows it, else the SIMT kernel */
    FD_ATTN_SIMT = 1,         /* CUDA-core split-KV kernel (any supported shape) */
    FD_ATTN_TCGEN05 = 2,      /* tcgen05 / TMEM / TMA split-KV kernel (head_dim 64 or 128); how it finds its work is
                                 chosen per call, see FD_TC_* */
    FD_ATTN_TCGEN05_PLANNED = 3,      /* the same kernel, always on the plan kernel's work list (FD_TC_PLANNED) */
    FD_ATTN_TCGEN05_SELF_PLANNED = 4  /* the same kernel, planning for itself wherever the call is small enough
                                         (FD_TC_SELF_PLANNED), never one cluster per segment */
};

/* How a call of the tensor-core attention kernel found its work (fd_attn_last_mode).  All three give the same
 * result to within rounding order; the choice is about fixed cost.
 *   FD_TC_PLANNED       a one-CTA plan kernel (or fd_plan_pin, once per step) cuts all KV tiles of the call into
 *                       one range per SM ("stream-K"); ranges that share a (sequence, kv-head) segment leave
 *                       partial results in scratch memory and the last to arrive merges them.
 *   FD_TC_SELF_PLANNED  at most 24 sequences with query blocks of at most 128 / G rows: every CTA makes the same
 *                       cut itself in its prologue; one launch, nothing to wait for.
 *   FD_TC_CLUSTER       at most 18 segments (batch 1-2 at 8 kv-heads, the paper's parallel-mode operating point):
 *                       one thread-block cluster of up to 16 CTAs per segment splits its tiles evenly and merges
 *                       through distributed shared memory; one launch, no scratch memory, no counters. */
enum { FD_TC_PLANNED = 0, FD_TC_SELF_PLANNED = 1, FD_TC_CLUSTER = 2 };

typedef struct {
    int n_q_heads;            /* Hq */
    int n_kv_heads;           /* Hkv, divides Hq */
    int head_dim;             /* d: 64 or 128 */
    int page_size;            /* P: 16 */
    int vocab;                /* V >= 1 */
    int max_batch;            /* largest B of any call; at most 4096 */
    int max_q_len;            /* largest Lq_b, <= 4096.  Up to 128 / G block rows share one 128-row MMA tile; a
                                 longer query block is processed as several such row blocks, each streaming
                                 the sequence's KV on its own (the O(N^2) regime of preparing every hypothesis) */
    int max_pages_per_seq;    /* row length of page_table */
    float softmax_scale;      /* 0 selects 1/sqrt(d) */
    int attn_path;            /* FD_ATTN_* */
} fd_config;

/* Create a context on the current CUDA device.  Allocates all scratch memory: about 20 MB for
 * the attention (split partials, work list) plus, for the vocabulary sweeps, about 30 bytes per
 * (row, 4096-logit chunk) with max_batch * max_q_len rows -- 2 MB at batch 64, 32 rows and a
 * 152k vocabulary; size max_batch and max_q_len for the job.  *ctx is NULL on failure
 * (FD_ERR_WORKSPACE if the device has no room). */
fd_status fd_create(fd_ctx** ctx, const fd_config* cfg);

/* Free a context.  Synchronises the device first.  NULL is accepted. */
fd_status fd_destroy(fd_ctx* ctx);

/*
 * Attention of one target forward pass over the ragged query blocks (Sec. 4.1,
 * "Inference"; hybrid mask of Sec. 4.1 and the Fig. 2 caption).  For sequence b, q-head
 * h, block row i:
 *
 *     out[row0_b + i, h, :] = sum_{j in A_b(i)} softmax_j( scale * <q[row0_b+i, h], K_b[j, h/G]> ) V_b[j, h/G]
 *
 *     A_b(i), i <  C_b (candidate row): { j < n_b } U { n_b + t : t <= i }        causal; no mask token
 *     A_b(i), i >= C_b (mask row):      { j < kv_len_b }                          prefix, all candidates,
 *                                                                                 whole mask block
 *     K_b[j], V_b[j] = kv_cache[ page_table[b][j / P], 0 | 1, h / G, j % P, : ]
 *
 * The caller has already written K/V of all Lq_b query tokens (candidates first, then
 * mask tokens) at logical positions n_b .. n_b + Lq_b - 1 ("append, then attend"), with
 * positional encoding and norms applied.  Slots that no valid token owns may hold any
 * bit pattern (NaN included); they never influence the result.
 *
 *   batch          B, 0 <= B <= max_batch (B = 0 is a no-op)
 *   total_q_rows   T; must equal sum_b q_lens[b]
 *   q              device, [T, Hq, d] bf16, 16-byte aligned, sequence-major rows
 *   kv_cache       device, [num_pages, 2, Hkv, P, d] bf16, 128-byte aligned
 *   num_pages      size of the page pool
 *   page_table     device, [B, max_pages_per_seq] int32; entries beyond ceil(kv_len_b/P) are ignored
 *   prefix_lens, q_lens, n_mask   device, [B] int32
 *   out            device, [T, Hq, d] bf16, 16-byte aligned; fully overwritten
 *   stream         cudaStream_t
 *
 * Device-detected errors: a sequence with a page id outside the pool gets zeros in its
 * out rows (FD_DEV_BAD_PAGE); inconsistent lengths zero all T rows (FD_DEV_BAD_LENGTHS).
 * Arithmetic: bf16 inputs, fp32 scores / softmax / accumulation, bf16 output.
 */
fd_status fd_attn_draft_verify(fd_ctx* ctx, int batch, int total_q_rows,
                               const void* q, const void* kv_cache, int num_pages,
                               const int32_t* page_table, const int32_t* prefix_lens,
                               const int32_t* q_lens, const int32_t* n_mask,
                               void* out, void* stream);

/*
 * Optional: pin the work list of a step.  The attention call derives a work list (which CTA streams which
 * KV tiles) from the lengths alone; it is the same for every layer of a step.  fd_plan_pin computes it once;
 * until fd_plan_unpin, every fd_attn_draft_verify[_blocks] call with the same batch, total_q_rows and the
 * same four length pointers reuses it instead of recomputing it (a call with anything else that needs the plan
 * kernel recomputes and drops the pin; calls that plan for themselves, FD_TC_SELF_PLANNED and FD_TC_CLUSTER,
 * leave it alone).  The caller must not change the contents of the length arrays or of the page table while the
 * pin holds (from the second call it serves on, the kernel looks up its work and its first pages while the launch
 * before it on the stream is still running), and must unpin after a FD_DEV_TIMEOUT status (fd_last_device_status does so
 * itself when it reports that bit).  fd_kv_commit rewrites prefix_lens and therefore drops the pin
 * itself: the first attention call of the next step plans afresh (or is preceded by a new fd_plan_pin).
 * fd_kv_append leaves the lengths alone and keeps the pin.
 * Consecutive attention calls under one pin overlap on the device (fd_calls_back_to_back): a call starts while the call before it is still
 * finishing, and -- where its range of KV tiles is short -- reads its q and its cache ahead of that call's completion,
 * provided no earlier call since the pin wrote them (the library compares the `out` ranges of those calls with q and
 * kv_cache of this one; behind fd_kv_append, which writes the query block's own slots of the cache, the tiles that
 * lie wholly in the prefix are still read ahead, the ones that reach into the block after the append has completed).  fd_kv_append itself, behind an attention call of the chain, copies while that call finishes (its k_new /
 * v_new are checked against those `out` ranges in the same way).  Every write of an attention call (out, scratch)
 * waits for the launch before it, and the append waits for it before it ends, so results are those of calls run one
 * after the other.  What the library cannot see is a buffer written by the CALLER's own asynchronous work on another
 * stream: order such work before the call as usual.
 * The calls served by a pin must be ordered after fd_plan_pin (the
 * same stream, or streams the caller has ordered) and must not overlap one another: they share the context's
 * scratch memory, as all attention calls on one context do.
 * The paper does not describe a work list; this follows from "all layers of a step share the lengths".
 *
 *   prefix_lens, q_lens, n_mask   device, [B] int32;  n_blocks   device, [B] int32 or NULL
 */
fd_status fd_plan_pin(fd_ctx* ctx, int batch, int total_q_rows, const int32_t* prefix_lens, const int32_t* q_lens,
                      const int32_t* n_mask, const int32_t* n_blocks, void* stream);
fd_status fd_plan_unpin(fd_ctx* ctx);

/*
 * A whole step on device buffers in one call: for every layer the KV append (if k_new / v_new are given) and the
 * attention, on one work list (fd_plan_pin), then fd_verify_accept and fd_kv_commit -- the sequence of Sec. 4.1
 * "Inference" / Sec. 3, launched from C with nothing between the launches, so that consecutive calls overlap as under
 * fd_calls_back_to_back.  Everything a layer-by-layer caller gets from the single calls, this gives bit for bit.
 *
 *   q, k_new, v_new, kv_caches, out   HOST arrays of n_layers DEVICE pointers (k_new and v_new both NULL: no append);
 *                                     shapes per layer as fd_attn_draft_verify_blocks / fd_kv_append
 *   page_table, prefix_lens           device, in/out (the commit rewrites them)
 *   everything else                   device, as in the single calls; n_blocks may be NULL
 *
 * Asynchronous on `stream` like the single calls; errors as theirs (the first one is returned, later launches of the
 * step are skipped).
 */
fd_status fd_step_device(fd_ctx* ctx, int batch, int total_q_rows, int total_cand_rows, int n_layers,
                         const void* const* q, const void* const* k_new, const void* const* v_new,
                         void* const* kv_caches, void* const* out, int num_pages, int32_t* page_table,
                         int32_t* prefix_lens, const int32_t* q_lens, const int32_t* n_mask, const int32_t* n_blocks,
                         const float* logits, const int32_t* draft_tokens, int32_t* accepted_len,
                         int32_t* bonus_token, int32_t* freed_pages, int32_t* n_freed, void* stream);

/*
 * The caller's promise that lets consecutive calls overlap (default: off).  While on, the caller launches nothing of
 * its own on the stream between two calls on this context (a call on another context counts as the caller's own) --
 * the calls are back to back, as the layers of a benchmark step are, or as they are where everything between two
 * attention calls is itself ordered before the first of them.  The library then knows that the launch before a call is its own, and what that launch writes: see
 * fd_plan_pin (attention calls read q and the cache ahead, fd_kv_append copies under the tail of the attention call
 * before it) and fd_verify_accept (its sweep, like those of fd_verify_accept_sample and fd_draft_select, runs under
 * the tail of the attention call right before it).  Off, every call
 * waits for the launch before it before it reads anything but the pinned plan, the lengths and the page table: a
 * kernel of the caller's between two calls may then be any kernel, one that releases its dependents early included.
 * fd_step_host and fd_step_host_append, which launch nothing but this library's kernels, behave as if it were on.
 */
fd_status fd_calls_back_to_back(fd_ctx* ctx, int on);

/*
 * Host-side view of the work split, for schedulers and tests: how fd_attn_draft_verify cuts the 128-token KV
 * tiles of a call (numbered sequence-major, then kv-head, then position) into n_ranges contiguous ranges, one
 * per CTA of the tensor-core kernel.  Ranges have equal cost, a segment (sequence, kv-head) counting its tiles
 * plus a fixed start-up charge; a small call leaves the last ranges empty.  Runs on the CPU, touches no GPU.
 * The paper does not describe a work split; this is this library's own.
 *
 *   prefix_lens, q_lens   HOST, [B] int32 (a sequence has ceil((n_b + Lq_b) / 128) tiles per kv-head, none if Lq_b = 0)
 *   range_start           HOST, [n_ranges + 1] int32, out: first tile of every range; [n_ranges] = all tiles
 */
fd_status fd_plan_ranges_host(int batch, int n_kv_heads, const int32_t* prefix_lens, const int32_t* q_lens,
                              int n_ranges, int32_t* range_start);

/*
 * KV append, the step before the attention ("append, then attend").  The forward pass that verifies the
 * drafts also produces K/V for the query block; they enter the paged cache at logical positions
 * n_b .. n_b + Lq_b - 1 (candidates first, then mask tokens), where fd_attn_draft_verify reads them and
 * where, after fd_kv_commit has kept the accepted part, every later step finds them (Sec. 4.1
 * "Inference": the KV cache of the clean prefix is reused by all later steps).
 *
 *   k_new, v_new   device, [T, Hkv, d] bf16, 16-byte aligned, sequence-major rows
 *   kv_cache       device, [num_pages, 2, Hkv, P, d] bf16, in/out; only the slots of the block are written
 *   page_table     device, [B, max_pages_per_seq] int32: pages for positions up to n_b + Lq_b - 1 must be allocated
 *   prefix_lens, q_lens   device, [B] int32
 *
 * A sequence whose rows would pass T or the page table is skipped (FD_DEV_BAD_LENGTHS); a slot whose page
 * id is outside the pool is skipped (FD_DEV_BAD_PAGE).
 */
fd_status fd_kv_append(fd_ctx* ctx, int batch, int total_q_rows, const void* k_new, const void* v_new,
                       void* kv_cache, int num_pages, const int32_t* page_table,
                       const int32_t* prefix_lens, const int32_t* q_lens, void* stream);

/*
 * The same attention with several mask blocks per sequence: the parallel mode proper, in which the
 * forward pass that verifies the current draft also prepares one next-draft branch per hypothesis r
 * ("the first r drafts are accepted", Sec. 3 "Parallel speculative decoding", Eq. 2), each branch
 * conditioned on the prefix and on those r drafts only.
 *
 *   n_blocks   device, [B] int32, or NULL (= fd_attn_draft_verify).  nb_b = n_blocks[b]; 0 and 1 mean one
 *              block.  For nb_b > 1 the M_b mask rows are nb_b consecutive blocks of M_b / nb_b tokens
 *              (M_b divisible by nb_b, nb_b <= C_b); block g is the branch of hypothesis
 *              r = C_b - nb_b + g, so nb_b = C_b prepares every hypothesis r = 0..k_b.
 *
 *     A_b(i) for a mask row of block g:  { j < n_b } U { n_b + t : t <= r }  U  { its own block }
 *
 * (candidate row 0 is the known bonus token, candidate t the t-th draft); blocks never see each
 * other; candidate rows are as in fd_attn_draft_verify.  A query block may be as long as max_q_len
 * (the paper's full form, bonus + 16 drafts and 17 branches of 16 tokens, is 289 rows): 128 / G block
 * rows share one MMA tile per kv-head, a longer block is processed in several such row blocks.
 * Lengths that break the rules above zero all T rows (FD_DEV_BAD_LENGTHS).
 */
fd_status fd_attn_draft_verify_blocks(fd_ctx* ctx, int batch, int total_q_rows,
                                      const void* q, const void* kv_cache, int num_pages,
                                      const int32_t* page_table, const int32_t* prefix_lens,
                                      const int32_t* q_lens, const int32_t* n_mask,
                                      const int32_t* n_blocks, void* out, void* stream);

/*
 * Draft-side tail of the step (Sec. 4.2, Eq. 4; Sec. 4.3 "Selective verification", Eq. 5).  One row of
 * draft logits per mask token, sequence-major.  Calibrated logits l~ = l + bias (the bias is the output of
 * the calibration MLP of Eq. 4, evaluated by the caller; NULL = no calibration); the drafted token of a
 * row is argmax l~ (lowest index on ties, inputs NaN-free), its confidence p = softmax(l~)[token].  Within
 * every next-draft block (nb_b equal blocks per sequence, as in fd_attn_draft_verify_blocks) the cumulative
 * confidence of position i is prod_{r <= i} p_r -- Eq. 5's estimate of P(L_acc >= i) -- and keep_len of the
 * block is the number of leading positions where it is still >= threshold: how many of that branch's
 * drafts the next step should verify (its candidate rows are then 1 + keep_len).
 *
 *   total_mask_rows  Rm; must equal sum_b n_mask[b]
 *   max_blocks       row length of keep_len; every nb_b must be <= max_blocks
 *   draft_logits     device, [Rm, V] fp32            bias   device, [Rm, V] fp32, or NULL
 *   n_mask, n_blocks device, [B] int32 (n_blocks may be NULL)
 *   threshold        >= 0
 *   mask_tokens      device, [Rm] int32, written     mask_probs   device, [Rm] fp32, written
 *   keep_len         device, [B, max_blocks] int32, written (0 where a sequence has fewer blocks)
 *
 * Arithmetic: l + bias, the maxima and the confidences in fp32 (the sum of exponentials is accumulated in a
 * fixed order, so results are run-to-run identical).  Inconsistent lengths: tokens -1, confidences 0,
 * keep_len 0, FD_DEV_BAD_LENGTHS.
 */
fd_status fd_draft_select(fd_ctx* ctx, int batch, int total_mask_rows, int max_blocks,
                          const float* draft_logits, const float* bias,
                          const int32_t* n_mask, const int32_t* n_blocks, float threshold,
                          int32_t* mask_tokens, float* mask_probs, int32_t* keep_len, void* stream);

/*
 * Branch selection (Sec. 3: once verification has fixed r_acc, the branch prepared under that
 * hypothesis is the next draft).  mask_tokens holds one proposed token per mask row, sequence-major
 * ([sum_b M_b] int32, device).  For each sequence the block g = accepted_len[b] - (C_b - nb_b) is copied to
 * next_draft[b, 0:kb] (device, [B, max_block_len] int32, padded with -1) and next_len[b] = kb; when that
 * hypothesis was not prepared (g outside [0, nb_b)), the sequence has no mask rows, or
 * accepted_len[b] < 0, next_len[b] = 0.  A block longer than max_block_len raises FD_DEV_BAD_LENGTHS.
 */
fd_status fd_select_branch(fd_ctx* ctx, int batch, int max_block_len, const int32_t* mask_tokens,
                           const int32_t* q_lens, const int32_t* n_mask, const int32_t* n_blocks,
                           const int32_t* accepted_len, int32_t* next_draft, int32_t* next_len, void* stream);

/*
 * Lossless verification at temperature 0 (Sec. 3: draft tokens are accepted up to the
 * first rejection, the token produced there is the bonus token, committed length
 * L_acc = r_acc + 1).  With am[r] = argmax_v logits[r, v] (larger value wins, equal
 * values: lower index wins; inputs must be NaN-free) and r0_b the first candidate row of
 * sequence b:
 *
 *     accepted_len[b] = number of leading j < k_b with am[r0_b + j] == draft_tokens[r0_b + j + 1]
 *     bonus_token[b]  = am[r0_b + accepted_len[b]]
 *
 * so 0 <= accepted_len[b] <= k_b = C_b - 1 (this is the paper's r_acc).  A sequence with
 * C_b = 0 gets accepted_len = bonus_token = -1.
 *
 *   total_cand_rows  R; must equal sum_b (q_lens[b] - n_mask[b])
 *   logits           device, [R, V] fp32, candidate rows only, sequence-major
 *   draft_tokens     device, [R] int32: the token fed at each candidate row (row 0 of a
 *                    sequence is the previous bonus token and is never compared)
 *   q_lens, n_mask   device, [B] int32
 *   accepted_len, bonus_token   device, [B] int32, overwritten
 *
 * Inconsistent lengths: every accepted_len / bonus_token is set to -1 (FD_DEV_BAD_LENGTHS).
 * Right behind an attention call of the same context (fd_calls_back_to_back) the sweep over the logits starts while that
 * call is still finishing (neither reads what the other writes); the results are written after it has completed.
 */
fd_status fd_verify_accept(fd_ctx* ctx, int batch, int total_cand_rows,
                           const float* logits, const int32_t* draft_tokens,
                           const int32_t* q_lens, const int32_t* n_mask,
                           int32_t* accepted_len, int32_t* bonus_token, void* stream);

/*
 * Verification at temperature > 0 by speculative sampling (Sec. 3: whether a draft is kept depends on how
 * the target's probability p of the drafted token compares with the drafter's q; where the first draft is
 * dropped, the bonus token is drawn from what is left of p once q is taken out; committed length = accepted + 1).
 * Rows and draft_tokens as in fd_verify_accept.  With p_j = softmax(logits[row j] / T) and q_j =
 * softmax(draft_logits[row j] / T), draft j + 1 = x is accepted iff u_accept[row j] < min(1, p_j(x) / q_j(x));
 * rejected at j: bonus ~ max(0, p_j - q_j) normalised; all k accepted: bonus ~ p_k.  A token is drawn from
 * weights w by inverting their cumulative sum in index order at u_bonus[b] * sum(w).
 *
 *   logits        device, [R, V] fp32: target logits of the candidate rows
 *   draft_logits  device, [R, V] fp32 or NULL: row r holds the (calibrated) draft logits the token fed at row
 *                 r + 1 was proposed from; NULL = the drafter put all its mass on the proposed token
 *   temperature   > 0
 *   u_accept      device, [R] fp32 in [0, 1): one uniform per candidate row (a sequence's last row: unused)
 *   u_bonus       device, [B] fp32 in [0, 1)
 *   accepted_len, bonus_token   device, [B] int32, out; -1 for a sequence without candidate rows
 *
 * Probabilities are formed in fp32; a decision whose two sides differ by less than fp32 rounding may fall
 * either way.  Lengths that do not add up to R raise FD_DEV_BAD_LENGTHS.
 */
fd_status fd_verify_accept_sample(fd_ctx* ctx, int batch, int total_cand_rows, const float* logits,
                                  const float* draft_logits, const int32_t* draft_tokens, const int32_t* q_lens,
                                  const int32_t* n_mask, float temperature, const float* u_accept,
                                  const float* u_bonus, int32_t* accepted_len, int32_t* bonus_token, void* stream);

/*
 * KV commit / rollback.  The paper implies it (the clean-prefix KV cache is reused by
 * every later step, Sec. 4.1 "Inference" and Sec. 4.3 "Decoupled execution"; mask tokens
 * are invisible to clean tokens) without spelling it out; the reading implemented: the
 * bonus row and the accepted drafts stay, every later position of the block (rejected
 * drafts, mask tokens) is dropped by truncating the length and releasing the pages that
 * no kept token lives in.  For b ascending, with new_len = n_b + accepted_len[b] + 1:
 *
 *     for p = ceil(new_len / P) .. ceil((n_b + Lq_b) / P) - 1 ascending:
 *         append page_table[b][p] to freed_pages; page_table[b][p] = -1
 *     prefix_lens[b] = new_len
 *
 * KV bytes are not touched.  Sequences with accepted_len[b] < 0 are left unchanged; one with
 * accepted_len[b] >= q_lens[b] is left unchanged and raises FD_DEV_BAD_ACCEPT.
 *
 *   page_table    device, [B, max_pages_per_seq] int32, in/out
 *   prefix_lens   device, [B] int32, in/out
 *   q_lens, accepted_len   device, [B] int32
 *   freed_pages   device, int32, capacity >= B * (ceil(max_q_len / P) + 1), packed output
 *   n_freed       device, [1] int32, output
 */
fd_status fd_kv_commit(fd_ctx* ctx, int batch, int32_t* page_table, int32_t* prefix_lens,
                       const int32_t* q_lens, const int32_t* accepted_len,
                       int32_t* freed_pages, int32_t* n_freed, void* stream);

/*
 * One whole decode step from HOST buffers: the attention of n_layers layers, the verification
 * and the commit (the three calls above, in the order of Sec. 4.1 "Inference"), with every
 * per-step input copied up and every result copied back by the library.  The KV caches are
 * decode state and stay on the device; all other pointers are host pointers (pinned memory
 * makes the copies asynchronous and lets them overlap the kernels; pageable memory works but
 * serialises).  Copies run on two internal streams so that q of layer l+1 goes up and out of
 * layer l-1 comes back while layer l computes; one cudaMemcpyAsync per buffer.
 *
 * fd_host_reserve(ctx, max_total_q_rows, max_total_cand_rows) allocates the device staging
 * (2 x q, 2 x out, 2 x the block's K and V, logits, small arrays) and the copy streams once; it is the only part that
 * allocates and must precede fd_step_host.  A second call with sizes within the first is a
 * no-op; larger sizes return FD_ERR_INVALID_ARG.
 *
 *   kv_caches         host array of n_layers device pointers, each [num_pages, 2, Hkv, P, d] bf16
 *   q_host            [n_layers][T, Hq, d] bf16          out_host   [n_layers][T, Hq, d] bf16, written
 *   logits_host       [R, V] fp32                        draft_tokens_host [R] int32
 *   page_table_host   [B, max_pages_per_seq] int32, in/out (the commit's edits come back)
 *   prefix_lens_host  [B] int32, in/out                  q_lens_host, n_mask_host [B] int32
 *   n_blocks_host     [B] int32 mask blocks per sequence (see fd_attn_draft_verify_blocks), or NULL
 *   accepted_len_host, bonus_token_host [B] int32, written
 *   freed_pages_host  capacity B * (ceil(max_q_len / P) + 1) int32, written; n_freed_host [1]
 *
 * The call returns after enqueueing; `stream` has finished the step, results on the host
 * included, once everything enqueued on it has completed.  The host buffers must stay valid
 * and untouched until then.  Steps on one context must not overlap.
 */
fd_status fd_host_reserve(fd_ctx* ctx, int max_total_q_rows, int max_total_cand_rows);
fd_status fd_step_host(fd_ctx* ctx, int batch, int total_q_rows, int total_cand_rows, int n_layers,
                       const void* const* kv_caches, int num_pages, const void* q_host, void* out_host,
                       const float* logits_host, const int32_t* draft_tokens_host,
                       int32_t* page_table_host, int32_t* prefix_lens_host,
                       const int32_t* q_lens_host, const int32_t* n_mask_host,
                       const int32_t* n_blocks_host,
                       int32_t* accepted_len_host, int32_t* bonus_token_host,
                       int32_t* freed_pages_host, int32_t* n_freed_host, void* stream);

/*
 * The same step with the KV append inside (Sec. 4.1 "Inference": the K/V that the target's own forward pass
 * computes for the query block go into the cache, where this step's attention and every later step find them).
 * Per layer the block's K/V go up with its q, fd_kv_append writes them into the layer's pages, and the attention
 * call follows on the same stream under programmatic dependent launch (its set-up overlaps the append's tail).
 *
 *   k_new_host, v_new_host   [n_layers][T, Hkv, d] bf16, rows sequence-major as q; both NULL = fd_step_host
 *   kv_caches                as above, but written: positions n_b .. n_b + Lq_b - 1 of every sequence
 */
fd_status fd_step_host_append(fd_ctx* ctx, int batch, int total_q_rows, int total_cand_rows, int n_layers,
                              void* const* kv_caches, int num_pages, const void* q_host, const void* k_new_host,
                              const void* v_new_host, void* out_host, const float* logits_host,
                              const int32_t* draft_tokens_host, int32_t* page_table_host, int32_t* prefix_lens_host,
                              const int32_t* q_lens_host, const int32_t* n_mask_host, const int32_t* n_blocks_host,
                              int32_t* accepted_len_host, int32_t* bonus_token_host, int32_t* freed_pages_host,
                              int32_t* n_freed_host, void* stream);

/*
 * fd_verify_accept without any allocation.  (The paper has no counterpart; this entry point
 * exists for the callers described here.)
 *
 * Who needs it: code that must not call cudaMalloc -- a plugin running inside a serving
 * process whose memory pool owns every byte of the device, a step that runs while a CUDA
 * graph is being captured elsewhere in the process, a late-initialised worker that finds the
 * device already full.  fd_create() is closed to such callers because it allocates the
 * context's scratch memory.  This call needs no context: the (value, index) maxima of the
 * vocabulary sweep and the finished-CTA counter live in a fixed array compiled into the
 * library (FD_STATIC_MAX_ROWS * 8 bytes + 64 bytes = 32.06 KB of device memory on every GPU
 * that loads the library, held until the process exits).
 *
 * Semantics, argument layout and results are those of fd_verify_accept, with these changes:
 *   vocab           V, passed per call (there is no fd_config)
 *   device_status   device pointer to one int32 that receives FD_DEV_* bits (OR-ed in; the
 *                   caller clears it), or NULL to drop them
 * Limits: total_cand_rows <= FD_STATIC_MAX_ROWS and batch <= FD_STATIC_MAX_BATCH, else
 * FD_ERR_STATIC_LIMIT is returned and nothing is launched.
 *
 * The call allocates nothing: no cudaMalloc / cudaFree, no allocating library routine; it
 * enqueues two small cudaMemsetAsync (the part of the array it is about to use keeps the
 * previous call's contents and must start at zero) and one kernel on `stream`.
 * First call on each device: the device address of the array is looked up once
 * (cudaGetSymbolAddress, with that device current) and cached; make that first call outside
 * any stream capture.
 * Every call in the process shares the one array per device.  Calls issued on one stream are
 * safe back to back; calls that can overlap on the GPU (different streams, different threads,
 * different contexts of the same library image) race on it and must be serialised by the caller.
 */
#define FD_STATIC_MAX_ROWS 4096
#define FD_STATIC_MAX_BATCH 4096
fd_status fd_verify_accept_static(int vocab, int batch, int total_cand_rows,
                                  const float* logits, const int32_t* draft_tokens,
                                  const int32_t* q_lens, const int32_t* n_mask,
                                  int32_t* accepted_len, int32_t* bonus_token,
                                  int32_t* device_status, void* stream);

/* Read and clear the sticky device status word (an OR of FD_DEV_* bits) into *code (host
 * pointer).  Synchronises `stream` first. */
fd_status fd_last_device_status(fd_ctx* ctx, int32_t* code, void* stream);

/* Failure-detection self-test (no counterpart in the paper).  Every device-side wait of the
 * attention kernel is bounded: when it runs out, the kernel stops cleanly and raises
 * FD_DEV_TIMEOUT instead of hanging the GPU.  This call exercises exactly that mechanism on a
 * barrier that nothing will ever signal: one warp waits for `limit_ms` (1..1000) milliseconds,
 * gives up, sets FD_DEV_TIMEOUT in the status word and returns.  The context stays usable. */
fd_status fd_selftest_wait_timeout(fd_ctx* ctx, int limit_ms, void* stream);

/* Which attention kernel the context resolved to: FD_ATTN_SIMT or FD_ATTN_TCGEN05. */
int fd_attn_path(const fd_ctx* ctx);

/* FD_TC_* of the context's most recent tensor-core attention call, -1 before the first one. */
int fd_attn_last_mode(const fd_ctx* ctx);

/* Number of CUDA kernels this library has launched through `ctx` since fd_create. */
int64_t fd_launch_count(const fd_ctx* ctx);

/* Static string for a status code. */
const char* fd_status_string(fd_status s);

#ifdef __cplusplus
}
#endif
#endif /* FLEXDRAFT_H */
