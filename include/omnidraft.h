/*
 * omnidraft.h — C ABI of the B200 (sm_100a) cross-vocabulary speculative
 * verification step of OmniDraft (arXiv 2507.02659).
 *
 * One verification step, per sequence b of a batch (Algorithm 1, from the
 * translation line to the free-token line):
 *   1. od_map_proposals   translate the K_b proposed draft tokens into m_b
 *                         target tokens t_i with draft probabilities q'(t_i)
 *                         through the direct vocabulary map and the n-gram
 *                         cache (Section 3.1, Eq. (1));
 *   2. od_verify          temperature softmax of the m_b + 1 target-logit
 *                         rows, acceptance ratio min(1, p(t_i)/q'(t_i)),
 *                         accepted prefix length n_b (Algorithm 1);
 *   3. od_sample_residual the extra token: drawn from norm(max(0, p - q'))
 *                         with q'(.) of Eq. (2) at the first rejection, or
 *                         from p (the free token) when everything was
 *                         accepted.
 *
 * Conventions
 *   - Every function returns an od_status (0 = OD_OK, negative = error). No
 *     exceptions, no aborts, no output on stdout/stderr.
 *   - "host" pointers are ordinary host memory read during the call.
 *     "device" pointers are global memory of the context's GPU, owned by the
 *     caller and neither retained nor freed by the library.
 *   - The three step functions are asynchronous on `stream` (a cudaStream_t
 *     passed as void*, NULL = the legacy default stream), allocate nothing and
 *     never synchronise. Arguments are validated on the host (scalars,
 *     alignment); data-dependent conditions are reported in device-side flag
 *     words, never by a trap.
 *   - A context holds scratch that its kernels share: calls on one context
 *     must be ordered (one stream, or explicit dependencies). Use one context
 *     per concurrent stream, and make the calls of one step on one context.
 *   - With option "pdl" = 1 (the default) the step kernels are launched with
 *     programmatic stream serialization: a kernel may become resident while
 *     the launch in front of it in the stream still runs, and executes
 *     griddepcontrol.wait before it touches anything that launch may write.
 *     What a kernel reads BEFORE its wait is only what the library itself can
 *     prove complete: outputs of a library kernel that finished before the
 *     kernel in front was allowed to start. Inputs of the caller (logits,
 *     temperatures, seeds, draft ids and probabilities) are read before the
 *     wait in two cases only: inside od_step / od_step_host, where the
 *     translation kernel is the launch in front of the streaming kernel and has
 *     itself waited for everything earlier in the stream before letting it
 *     start (logits and temperatures, by the streaming kernel); and when the
 *     caller has set option "early_inputs" = 1, which is the caller's promise
 *     that the inputs of a call were complete before the launch that precedes
 *     the call was enqueued (a producer two launches back, or data resident
 *     since an earlier synchronisation): then od_verify and
 *     od_verify_shard_stats read logits and temperatures early;
 *     od_map_proposals and od_step read the proposal (draft ids, lengths,
 *     q_sel) early and, unless od_cache_insert or od_cache_trim was called on
 *     the context since its last translation, probe the n-gram table early
 *     (the table belongs to the context; the library keeps track of who writes
 *     it); and od_step lets its streaming kernel start on logit rows 0 while the
 *     launch in front of the step still runs. What the library keeps track of
 *     it knows at the time of the call: a CUDA graph that captured
 *     od_map_proposals or od_step under "early_inputs" = 1 must not be launched
 *     directly behind od_cache_insert or od_cache_trim (any launch in between
 *     that is not programmatic, or an event, restores the order). A producer that is
 *     the launch directly in front of a call (the target model's output layer,
 *     the drafter's sampling kernel) is always safe with the default
 *     "early_inputs" = 0. od_step_host copies its inputs itself and reads
 *     nothing of the caller's early. "pdl" = 0 gives plain stream order.
 *   - Positions: arrays indexed [B, K_max] hold K_max entries per sequence,
 *     of which the first K_b (inputs) or m_b (outputs) are meaningful.
 *   - Random numbers: Philox4x32-10 (Salmon et al., SC'11) with key = the
 *     sequence's 64-bit seed and counter = (step lo, step hi, position, tag);
 *     u = (word0 >> 8) * 2^-24. tag 0 = acceptance test at `position`,
 *     tag 1 = extra-token draw at `position`.
 */
#ifndef OMNIDRAFT_H
#define OMNIDRAFT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct od_ctx od_ctx;

enum od_status {
    OD_OK = 0,
    OD_ERR_INVALID_ARG = -1,       /* NULL pointer, size out of range */
    OD_ERR_ALIGNMENT = -2,         /* logits base or stride not 16-byte aligned */
    OD_ERR_MAP_NOT_INJECTIVE = -3, /* two draft ids map to one target id */
    OD_ERR_BAD_CACHE_ENTRY = -4,   /* run length outside 2..4, id out of range */
    OD_ERR_UNSUPPORTED = -5,       /* dtype, vocabulary too large for the cache key */
    OD_ERR_CUDA = -6,              /* a CUDA runtime call failed */
    OD_ERR_NOMEM = -7,
    OD_ERR_STATE = -8,             /* call out of order (e.g. no vocabulary map yet) */
    OD_ERR_SCRATCH_LIMIT = -9      /* od_verify_noalloc: batch too large for its fixed scratch */
};

enum od_dtype { OD_F32 = 0, OD_BF16 = 1 };

/* tail_kind[b] written by od_map_proposals */
enum od_tail {
    OD_TAIL_COMPLETE = 0,      /* all K_b draft tokens were translated */
    OD_TAIL_UNMAPPED_STOP = 1  /* translation stopped at a token with neither a
                                  cache hit nor a direct map: position m_b is a
                                  forced rejection */
};

/* counters[] accumulated (atomically added to) by od_map_proposals */
enum od_counter {
    OD_CNT_CACHE_HITS = 0,
    OD_CNT_UNMAPPED_STOPS = 1,
    OD_CNT_INVALID_IDS = 2,    /* draft ids outside [0, draft_vocab) */
    OD_CNT_MAPPED_TOKENS = 3,  /* sum of m_b */
    OD_CNT_COUNT = 4
};

/* verify_flags[b] written by od_verify */
#define OD_VF_BOUNDARY_MASK 0x0000FFFFu /* bit i: |u_i - ratio_i| <= OD_TAU_ACCEPT */
#define OD_VF_BAD_TEMPERATURE 0x00010000u
#define OD_VF_NONFINITE 0x00020000u     /* a row sum is not finite and positive */

/* sample_flags[b] written by od_sample_residual */
#define OD_SF_BOUNDARY 0x1u        /* u*R within OD_TAU_SAMPLE*R of a CDF edge of the token */
#define OD_SF_ZERO_MASS 0x2u       /* residual mass <= 0: drawn from p instead */
#define OD_SF_BAD_TEMPERATURE 0x4u
#define OD_SF_BONUS 0x10u          /* the token is the free token (n_b == m_b) */

/* fp32 arithmetic can land on the other side of a decision than exact
 * arithmetic only inside these margins; such decisions are flagged. */
#define OD_TAU_ACCEPT 1.0e-5f
#define OD_TAU_SAMPLE 2.0e-6
#define OD_TAU_EXIT 4.0e-6f

#define OD_MAX_K 16      /* largest K_max */
#define OD_NOALLOC_MAX_ROWS 1024 /* od_verify_noalloc: largest B * (K_max + 1) */
#define OD_NGRAM_MAX 4   /* longest cached run */

/* ---- context ----------------------------------------------------------- */

/* Create a context on CUDA device `device` for a draft vocabulary of
 * `draft_vocab` ids and a target vocabulary of `target_vocab` ids, for
 * batches of at most `max_batch` sequences with at most `max_k`
 * (1..OD_MAX_K) proposed tokens each. Allocates the device-side scratch
 * (tickets, partial row statistics, tile sums) once; synchronous.
 * target_vocab is bounded by what od_sample_residual keeps in shared memory
 * (8 bytes per 256 ids, at most 200 KB: 6,553,600 ids); larger vocabularies
 * are refused with OD_ERR_UNSUPPORTED. */
int32_t od_create(od_ctx **ctx, int32_t device, int32_t draft_vocab,
                  int32_t target_vocab, int32_t max_batch, int32_t max_k);

/* Free everything the context owns. Synchronises the device first. */
int32_t od_destroy(od_ctx *ctx);

/* Direct vocabulary map t <-> d on the intersection of the vocabularies
 * (Eq. (1), first case). host_map: int32[draft_vocab], target id or -1.
 * Builds the inverse map, uploads both (synchronous). Rejects target ids
 * outside [0, target_vocab) (INVALID_ARG) and maps that send two draft ids to
 * one target id (MAP_NOT_INJECTIVE). */
int32_t od_set_vocab_map(od_ctx *ctx, const int32_t *host_map);

/* n-gram cache C = {(t, [d_1..d_n])} (Section 3.1). host_runs: int32[E,4],
 * unused slots ignored; host_len: int32[E] in 2..4; host_target: int32[E].
 * Builds an open-addressing table (32-slot groups, load <= 1/2) on the host,
 * deterministically, and uploads it (synchronous). When a run appears twice
 * the first entry wins (Algorithm 1 only inserts an unseen n-gram). E = 0
 * installs an empty cache. Replaces any earlier cache. Needs
 * draft_vocab <= 65535 when E > 0 (UNSUPPORTED otherwise): a run is packed
 * into one 64-bit key, 16 bits per id. */
int32_t od_cache_build(od_ctx *ctx, const int32_t *host_runs,
                       const int32_t *host_len, const int32_t *host_target,
                       int64_t E);

/* ---- online cache -------------------------------------------------------- */

/* The cache as Algorithm 1 grows it (cache-update line: an n-gram that is not in
 * the cache yet is added) and bounds it (App. D.5: a maximum size with LRU, which
 * evicts the n-gram not accessed for the longest time, or LFU, which evicts the one
 * with the lowest access frequency). Where the paper is silent: an access is a
 * cached run that od_map_proposals actually merges (and the insertion itself); time
 * is a clock the caller sets, one tick per verification step; eviction is an explicit
 * trim; ties go by the run's packed key; entries inserted at the current clock are
 * evicted last.
 *
 * od_cache_configure installs an EMPTY online cache for at most `max_entries`
 * entries after a trim (policy 0 = LRU, 1 = LFU) and batches of at most `max_insert`
 * candidates; it replaces any earlier cache (od_cache_build does the reverse) and is
 * synchronous. Needs draft_vocab <= 65535 (UNSUPPORTED otherwise). Device memory:
 * the table has S = the next power of two >= 2 * (max_entries + max_insert) slots;
 * two copies of it (24 bytes per slot each, the second one is the table a trim
 * builds), a claim word per slot and 68 bytes per slot of trim scratch are
 * allocated here, 120 * S bytes in all (NOMEM if that fails); nothing is
 * allocated later. */
int32_t od_cache_configure(od_ctx *ctx, int64_t max_entries, int32_t policy,
                           int32_t max_insert);

/* The clock that stamps accesses (od_map_proposals) and insertions enqueued from
 * now on. Host-side; STATE without an online cache. */
int32_t od_cache_set_clock(od_ctx *ctx, uint32_t clock);

/* Adds the candidates that are not in the cache yet. device: runs int32[N,4]
 * (draft ids, the first len[i] are used), len int32[N] in 2..4, target int32[N].
 * Of several candidates with the same run the one with the lowest index wins, as
 * if they were added one after the other; malformed candidates (length, ids or
 * target out of range) are skipped. New entries get the current clock as time of
 * insertion and of last access, and frequency 1. Asynchronous on `stream`; must be
 * ordered with od_map_proposals on the same context. N <= max_insert.
 * The table is sized for max_entries + max_insert entries at load 1/2: trim at
 * least once per batch that can take the cache past max_entries. A candidate that
 * finds no free slot on its whole probe sequence (only possible when trims were
 * skipped for many batches) is dropped and counted (od_cache_stats). */
int32_t od_cache_insert(od_ctx *ctx, int32_t N, const int32_t *runs,
                        const int32_t *len, const int32_t *target, void *stream);

/* If the cache holds k > 0 entries more than max_entries, drops the k entries that
 * come first in the order (inserted at the current clock? no before yes; then last
 * access clock for LRU or frequency for LFU, ascending; then the run's packed key,
 * ascending) and rebuilds the table. Asynchronous on `stream` (a fixed sequence of
 * small kernels, no host round trip); calls enqueued afterwards see the new table.
 * The table's address and the clock are arguments of the kernels that use them: a
 * CUDA graph that captured od_map_proposals (or od_step) keeps the table and the
 * clock of its capture and must be captured again after od_cache_trim or
 * od_cache_set_clock. */
int32_t od_cache_trim(od_ctx *ctx, void *stream);

/* Counters of the online cache since od_cache_configure (synchronises the device; any
 * pointer may be NULL): the number of entries; the malformed candidates od_cache_insert
 * skipped; the candidates it lost because their whole probe sequence was full, which
 * happens only when trims were skipped for so long that the table filled up (Algorithm 1's
 * cache update has no such case: the paper's cache is unbounded unless trimmed, App. D.5).
 * STATE without an online cache. */
int32_t od_cache_stats(od_ctx *ctx, int64_t *entries, int64_t *invalid, int64_t *dropped);

/* Contents of the online cache, for inspection and tests: synchronises the device,
 * writes up to max_out entries (host arrays: runs int32[max_out,4] padded with -1,
 * len, target, and, if not NULL, the last-access clock and the frequency) in no
 * particular order, and the total number of entries to *n_out. */
int32_t od_cache_dump(od_ctx *ctx, int64_t max_out, int32_t *runs, int32_t *len,
                      int32_t *target, uint32_t *stamp, uint32_t *freq, int64_t *n_out);

/* Options. Names: "pdl" (1 = launch the step kernels with programmatic stream
 * serialization so that a kernel's prologue overlaps its predecessor's tail, the
 * default; 0 = plain stream order), "early_inputs" (1 = od_verify and
 * od_verify_shard_stats may read logits and temperatures, od_map_proposals and
 * od_step the proposal, before they wait for the launch in front of them, see the
 * conventions above; default 0),
 * "verify_grid" (thread blocks of od_verify's streaming kernel, 0 = one per
 * multiprocessor, the default), "sample_tiles_per_warp" (256-id tiles one warp of
 * od_sample_residual sums, 0 = automatic). Unknown name: INVALID_ARG. */
int32_t od_set_option(od_ctx *ctx, const char *name, int64_t value);

/* ---- the step ----------------------------------------------------------- */

/* Step 1 (Eq. (1); Algorithm 1, translation line). Scan d_0..d_{K_b-1} left to
 * right; at each offset try the cached runs of length min(4, remaining)..2,
 * longest first; on a hit emit (t, prod_j q(d_j)) and skip the run; otherwise
 * emit the directly mapped token (map[d], q(d)); a token with neither ends the
 * translation (OD_TAIL_UNMAPPED_STOP).
 *   in  (device) draft_ids  int32[B,K_max]   proposed draft ids
 *                draft_len  int32[B]         K_b, clamped to [0, K_max]
 *                q_sel      float[B,K_max]   q(d_j) of each proposed token
 *   out (device) tgt_ids    int32[B,K_max]   t_i, i < m_b
 *                q_prime    float[B,K_max]   q'(t_i), i < m_b
 *                span_start int32[B,K_max]   first draft position of piece i;
 *                                            under UNMAPPED_STOP entry m_b is
 *                                            the stopping position
 *                span_len   int32[B,K_max]   draft tokens merged into piece i
 *                m          int32[B]         number of translated tokens
 *                tail_kind  uint8[B]         enum od_tail
 *                counters   uint32[OD_CNT_COUNT], added to (may be NULL)
 * Entries at positions >= m_b (beyond the stop entry) are left untouched. */
int32_t od_map_proposals(od_ctx *ctx, int32_t B, int32_t K_max,
                         const int32_t *draft_ids, const int32_t *draft_len,
                         const float *q_sel, int32_t *tgt_ids, float *q_prime,
                         int32_t *span_start, int32_t *span_len, int32_t *m,
                         uint8_t *tail_kind, uint32_t *counters, void *stream);

/* Step 2 (Algorithm 1, target-probability and rejection lines). For each
 * sequence, rows 0..m_b of its logits are read exactly once:
 * M_r = max_t x_t, S_r = sum_t exp((x_t - M_r)/T_b); for i < m_b
 * p_sel_i = exp((x[t_i] - M_i)/T_b)/S_i, ratio_i = 1 if q'_i <= p_sel_i else
 * p_sel_i/q'_i, accepted iff u_i < ratio_i; n_b = number of leading accepts.
 *   in  (device) logits  fp32 or bf16, element (b, r, t) at
 *                        b*seq_stride + r*row_stride + t (strides in elements);
 *                        base and both strides must be multiples of 16 bytes;
 *                        rows above m_b are never touched
 *                tgt_ids, q_prime, span_len, m  as written by step 1
 *                temperature float[B] (> 0, else BAD_TEMPERATURE is flagged
 *                        and n_b = 0), seed uint64[B]
 *   out (device) row_max, row_sum float[B,K_max+1]   rows 0..m_b
 *                p_sel, ratio    float[B,K_max]      i < m_b
 *                n_accepted, n_draft_accepted int32[B] (the latter = draft
 *                        tokens covered by the accepted pieces)
 *                verify_flags uint32[B] */
int32_t od_verify(od_ctx *ctx, int32_t B, int32_t K_max, const void *logits,
                  int32_t logit_dtype, int64_t row_stride, int64_t seq_stride,
                  const int32_t *tgt_ids, const float *q_prime,
                  const int32_t *span_len, const int32_t *m,
                  const float *temperature, const uint64_t *seed, uint64_t step,
                  float *row_max, float *row_sum, float *p_sel, float *ratio,
                  int32_t *n_accepted, int32_t *n_draft_accepted,
                  uint32_t *verify_flags, void *stream);

/* Step 3 (notation paragraph of Section 3: residual; Eq. (2); Algorithm 1,
 * rejection and free-token lines). Position j = n_b. If j < m_b, or j == m_b
 * under UNMAPPED_STOP: r(t) = max(0, p_j(t) - q'_j(t)) where q'_j(.) is the
 * drafter's row q_rows[b, span_start_j, .] carried through the inverse map (0
 * outside the map's image), and, when piece j is a cached n-gram with token T
 * and first sub-token d_1: q'_j(map[d_1]) = q(d_1) - q'(T) (if d_1 is mapped)
 * and then q'_j(T) = q'(T). Otherwise (free token) r = p_m. The output is the
 * smallest t whose inclusive cumulative sum exceeds u*R, R = sum_t r(t), in
 * target-id order. If R <= 0 the token is drawn from p_j and ZERO_MASS is set.
 *   in  (device) logits (as for od_verify), row_max, row_sum from step 2,
 *                q_rows float[B,K_max,draft_vocab] drafter distributions,
 *                draft_ids, tgt_ids, q_prime, span_start, span_len, m,
 *                tail_kind from step 1, n_accepted from step 2,
 *                temperature, seed, step as for step 2
 *   out (device) out_token int32[B], resid_mass float[B] (R),
 *                sample_flags uint32[B] */
int32_t od_sample_residual(od_ctx *ctx, int32_t B, int32_t K_max,
                           const void *logits, int32_t logit_dtype,
                           int64_t row_stride, int64_t seq_stride,
                           const float *row_max, const float *row_sum,
                           const float *q_rows, const int32_t *draft_ids,
                           const int32_t *tgt_ids, const float *q_prime,
                           const int32_t *span_start, const int32_t *span_len,
                           const int32_t *m, const uint8_t *tail_kind,
                           const int32_t *n_accepted, const float *temperature,
                           const uint64_t *seed, uint64_t step,
                           int32_t *out_token, float *resid_mass,
                           uint32_t *sample_flags, void *stream);

/* Steps 1-3 in one call (Algorithm 1 from the translation line to the free-token
 * line): exactly od_map_proposals, od_verify and od_sample_residual on the same
 * arguments, enqueued back to back on `stream`. Besides saving two calls, this is
 * the form in which the library knows its own launch order, so the streaming
 * kernel may start on rows 0 of the logits while the translation kernel still
 * runs, with no promise needed from the caller (see "pdl" in the conventions).
 * All pointers are device pointers owned by the caller; inputs and outputs as
 * documented for the three calls (counters may be NULL). Asynchronous; allocates
 * nothing; errors as for the three calls, checked before the first launch. */
int32_t od_step(od_ctx *ctx, int32_t B, int32_t K_max, const int32_t *draft_ids,
                const int32_t *draft_len, const float *q_sel, const float *q_rows,
                const void *logits, int32_t logit_dtype, int64_t row_stride,
                int64_t seq_stride, const float *temperature, const uint64_t *seed,
                uint64_t step, int32_t *tgt_ids, float *q_prime, int32_t *span_start,
                int32_t *span_len, int32_t *m, uint8_t *tail_kind, uint32_t *counters,
                float *row_max, float *row_sum, float *p_sel, float *ratio,
                int32_t *n_accepted, int32_t *n_draft_accepted, uint32_t *verify_flags,
                int32_t *out_token, float *resid_mass, uint32_t *sample_flags,
                void *stream);

/* Hybrid cross-vocabulary distillation loss (Section 3.2, Eq. (3)) of the proposals
 * of one verification step, per draft position j, and its gradient with respect to
 * the drafter's logits z (q = softmax(z)):
 *   j directly mapped (its piece has one sub-token, target position i):
 *       loss = KL(q' || p_i) = sum over mapped draft ids d of q(d) (ln q(d) - ln p_i(map[d])),
 *       grad(d) = q(d) (g(d) - sum_e q(e) g(e)),  g(d) = [d mapped] (ln q(d) - ln p_i(map[d]) + 1);
 *   j a sub-token of a cached n-gram:  loss = -w ln q(d_j),  grad(d) = w (q(d) - [d == d_j]),
 *       w = lambda (lambda_mode 0) or the verified target probability p_i(t_i) of the
 *       n-gram (lambda_mode 1, needs p_sel);
 *   j not translated (at or after an unmapped stop, beyond K_b) or T_b <= 0: 0.
 * p_i = softmax(row i / T_b), taken from the logits and from the row statistics that
 * od_verify wrote (row_max, row_sum). Sums over positions or the batch are the
 * caller's.
 *   in  (device) q_rows float[B,K_max,draft_vocab]; draft_ids; tgt_ids, span_start,
 *                span_len, m from od_map_proposals; logits, strides as for od_verify;
 *                row_max, row_sum, p_sel from od_verify; temperature float[B]
 *   out (device) loss float[B,K_max]; grad float[B,K_max,draft_vocab] (may be NULL)
 * Asynchronous on `stream`; allocates nothing. */
int32_t od_distill_loss(od_ctx *ctx, int32_t B, int32_t K_max, const float *q_rows,
                        const int32_t *draft_ids, const int32_t *tgt_ids,
                        const int32_t *span_start, const int32_t *span_len,
                        const int32_t *m, const void *logits, int32_t logit_dtype,
                        int64_t row_stride, int64_t seq_stride, const float *row_max,
                        const float *row_sum, const float *p_sel,
                        const float *temperature, float lambda, int32_t lambda_mode,
                        float *loss, float *grad, void *stream);

/* Adaptive drafting, exit rule (Section 3.3, Eq. (4)-(6)). From the acceptance
 * head's outputs f_phi(e_i) of the proposed tokens:
 *   reject_prob[b,k] = 1 - prod_{i<=k} sigmoid(head_logits[b,i])   (some token up
 *   to k is rejected), and draft_len[b] = the first k (1-based) at which that
 *   probability exceeds gamma, or avail_len[b] if it never does. The token whose
 *   test fires is part of the proposal. The head network itself is not part of
 *   this library.
 *   in  (device) head_logits float[B,K_max]; avail_len int32[B] tokens the drafter
 *                has produced per sequence, clamped to [0, K_max] (NULL = K_max);
 *                gamma in [0, 1] (INVALID_ARG otherwise)
 *   out (device) draft_len int32[B] (what od_map_proposals takes);
 *                reject_prob float[B,K_max], 0 at and beyond avail_len (may be NULL);
 *                exit_flags uint32[B], bit k: |reject_prob - gamma| <= OD_TAU_EXIT
 *                at a token up to the exit, where fp32 may decide differently
 *                from exact arithmetic (may be NULL).
 * Asynchronous on `stream`; allocates nothing. */
int32_t od_exit_rule(od_ctx *ctx, int32_t B, int32_t K_max, const float *head_logits,
                     const int32_t *avail_len, float gamma, int32_t *draft_len,
                     float *reject_prob, uint32_t *exit_flags, void *stream);

/* Step 2 without any allocation (the paper has no counterpart: this entry
 * point exists for the way some programs are built, not for the method).
 *
 * Who needs it: a caller that is handed its buffers and must not ask the CUDA
 * runtime for device memory itself. Typical cases are a plug-in inside a
 * serving process whose own allocator reserved the GPU's memory at start-up,
 * so a cudaMalloc from a library would fail or eat into memory the host
 * application budgeted, and a decode loop that cannot afford the device-wide
 * synchronisation cudaMalloc and cudaFree imply. Such a caller cannot use
 * od_create (which allocates the maps, the cache table and the kernels'
 * scratch), so this function takes no context: the target vocabulary size is an
 * argument, and it works on the CUDA device that is current when it is called.
 *
 * What it computes: exactly od_verify (same kernels, same arithmetic, same
 * outputs and flags; see above for the arguments, all device pointers owned by
 * the caller). What differs is the kernels' scratch, the per-segment partial
 * sums of the streaming pass: it is a fixed 1 MiB array compiled into the
 * library (OD_NOALLOC_MAX_ROWS rows x 64 partials x 16 bytes) that every GPU
 * loading the library holds until the process ends. The function calls no
 * cudaMalloc, cudaFree or other allocating routine. It always waits for the
 * launch in front of it before it reads the logits (there is no context to
 * carry the "early_inputs" promise), so any producer is safe.
 *
 * Limits and rules
 *   - B * (K_max + 1) <= OD_NOALLOC_MAX_ROWS and B <= 2048; anything larger is
 *     refused with OD_ERR_SCRATCH_LIMIT before any launch.
 *   - The first call on a device looks up the array's device address and the
 *     multiprocessor count (no allocation by this library, but host-side
 *     runtime calls). Where the CUDA runtime loads modules lazily, that first
 *     call is also the moment at which the driver loads the module and sets
 *     the array's 1 MiB aside, so free device memory can drop then, once.
 *     Make that first call during start-up, before any stream capture begins
 *     and before memory is tight.
 *   - All calls on a device share the one array. It keeps whatever the last
 *     call left in it; nothing in it needs clearing, because a call reads only
 *     the slots it has written itself. Two calls whose kernels overlap on the
 *     GPU (different streams, no dependency between them) race on it: order
 *     them. Calls on one stream are ordered.
 *   - Asynchronous on `stream` like od_verify; errors as for od_verify. */
int32_t od_verify_noalloc(int32_t target_vocab, int32_t B, int32_t K_max,
                          const void *logits, int32_t logit_dtype,
                          int64_t row_stride, int64_t seq_stride,
                          const int32_t *tgt_ids, const float *q_prime,
                          const int32_t *span_len, const int32_t *m,
                          const float *temperature, const uint64_t *seed,
                          uint64_t step, float *row_max, float *row_sum,
                          float *p_sel, float *ratio, int32_t *n_accepted,
                          int32_t *n_draft_accepted, uint32_t *verify_flags,
                          void *stream);

/* ---- whole step from host memory ---------------------------------------- */

/* Allocate device staging for od_step_host: inputs and outputs of one step of
 * max_batch x max_k, logits of `logit_dtype` stored densely. Synchronous. */
int32_t od_host_step_reserve(od_ctx *ctx, int32_t logit_dtype);

/* Steps 1-3 on HOST buffers (pinned memory recommended): copies the inputs to
 * the staging area, runs the three kernels, copies the results back, all on
 * `stream`, and synchronises that stream before returning. Host layouts are
 * the dense ones above (logits [B, K_max+1, target_vocab]); of the logits and
 * of q_rows only the rows the step can read are copied (rows 0..K_b and
 * 0..K_b-1 of sequence b, K_b = draft_len[b] read on the host). Outputs: host
 * int32[B] each for n_accepted, n_draft_accepted, out_token; int32[B,K_max]
 * tgt_ids; int32[B] m; uint32[B] verify_flags and sample_flags (any output may
 * be NULL). Needs od_host_step_reserve with the same dtype. */
int32_t od_step_host(od_ctx *ctx, int32_t B, int32_t K_max,
                     const int32_t *draft_ids, const int32_t *draft_len,
                     const float *q_sel, const float *q_rows,
                     const void *logits, int32_t logit_dtype,
                     const float *temperature, const uint64_t *seed,
                     uint64_t step, int32_t *n_accepted,
                     int32_t *n_draft_accepted, int32_t *out_token,
                     int32_t *tgt_ids, int32_t *m, uint32_t *verify_flags,
                     uint32_t *sample_flags, void *stream);

/* ---- the step with the target vocabulary split over GPUs ------------------ */

/* Steps 2 and 3 when the target model's output layer is split by columns over
 * n_shards GPUs (tensor parallelism): every GPU holds, for all rows, the logits of
 * the target ids [shard_lo, shard_lo + shard_len) only. The paper runs the target on
 * one GPU and has no counterpart of the split; the result is Algorithm 1's and
 * Eq. (2)'s, unchanged, because a row's softmax statistics and the residual's
 * cumulative sums are sums over disjoint id ranges. A step is
 *   od_verify_shard_stats   -> exchange (all-gather, the caller's) ->
 *   od_verify_shard_finish  -> od_sample_shard_mass -> exchange ->
 *   od_sample_shard_pick    -> exchange of the B picked tokens,
 * with the same od_map_proposals outputs, temperatures and seeds on every GPU, so
 * that all GPUs take identical decisions. Every context is created with the FULL
 * target vocabulary, map and cache. Shards must tile the vocabulary in id order;
 * shard_lo must be a multiple of 256 and shard_lo + shard_len either a multiple of
 * 256 or the vocabulary size (INVALID_ARG otherwise). `logits` points at the
 * shard's own buffer: element (b, r, shard_lo + c) at b*seq_stride + r*row_stride + c,
 * row_stride >= shard_len, alignment as for od_verify. All four calls are
 * asynchronous on `stream` and allocate nothing. */

/* Per-row statistics of this shard's columns (Algorithm 1, target-probability line,
 * restricted to the shard): stats[(b*(K_max+1) + r)*4 + 0..3] = (c, s, M, x) for rows
 * r <= m_b, where M is the exact maximum of the shard's logits of the row, c a
 * reference exponent in the scaled domain (c >= M*log2(e)/T_b up to rounding),
 * s = sum over the shard of exp2(x*log2(e)/T_b - c), and x = the logit of t_r if this
 * shard owns it (r < m_b), else -inf. Other rows are left untouched.
 *   in  (device) logits (the shard's), tgt_ids, m from od_map_proposals, temperature
 *   out (device) stats float[B*(K_max+1)*4], 16-byte aligned */
int32_t od_verify_shard_stats(od_ctx *ctx, int32_t B, int32_t K_max, int32_t shard_lo,
                              int32_t shard_len, const void *logits, int32_t logit_dtype,
                              int64_t row_stride, int64_t seq_stride,
                              const int32_t *tgt_ids, const int32_t *m,
                              const float *temperature, float *stats, void *stream);

/* Merges the records of all shards (stats_all = the n_shards stats arrays one after
 * the other, in shard order) and produces exactly the outputs of od_verify
 * (1 <= n_shards <= 1024). Deterministic: every GPU gets the same bits. */
int32_t od_verify_shard_finish(od_ctx *ctx, int32_t B, int32_t K_max, int32_t n_shards,
                               const float *stats_all, const int32_t *tgt_ids,
                               const float *q_prime, const int32_t *span_len,
                               const int32_t *m, const float *temperature,
                               const uint64_t *seed, uint64_t step, float *row_max,
                               float *row_sum, float *p_sel, float *ratio,
                               int32_t *n_accepted, int32_t *n_draft_accepted,
                               uint32_t *verify_flags, void *stream);

/* This shard's share of the mass the extra token is drawn from (arguments as for
 * od_sample_residual, row_max / row_sum / n_accepted from od_verify_shard_finish):
 * mass[2b] = sum over the shard's ids of r(t) (unnormalised: times the row sum),
 * mass[2b+1] = the shard's share of p_j in the same units if mass[2b] is zero for a
 * residual draw (needed when no shard has residual mass), else 0.
 *   out (device) mass double[B*2] */
int32_t od_sample_shard_mass(od_ctx *ctx, int32_t B, int32_t K_max, int32_t shard_lo,
                             int32_t shard_len, const void *logits, int32_t logit_dtype,
                             int64_t row_stride, int64_t seq_stride, const float *row_max,
                             const float *row_sum, const float *q_rows,
                             const int32_t *draft_ids, const int32_t *tgt_ids,
                             const float *q_prime, const int32_t *span_start,
                             const int32_t *span_len, const int32_t *m,
                             const uint8_t *tail_kind, const int32_t *n_accepted,
                             const float *temperature, double *mass, void *stream);

/* The draw, after the shares of all shards were exchanged (mass_all = the n_shards
 * mass arrays in shard order; must follow od_sample_shard_mass of the same step on
 * this context, which leaves the shard's tile sums in the context's scratch). The
 * inverse-CDF walk of od_sample_residual runs over the shards in id order and, inside
 * the shard it stops in, over that shard's ids. Exactly one shard writes the token:
 * the others write out_token = -1, resid_mass = 0, sample_flags = 0, so that the
 * element-wise maximum (tokens, masses) and OR (flags) over the shards is the result
 * of od_sample_residual. */
int32_t od_sample_shard_pick(od_ctx *ctx, int32_t B, int32_t K_max, int32_t n_shards,
                             int32_t shard_index, int32_t shard_lo, int32_t shard_len,
                             const double *mass_all, const void *logits,
                             int32_t logit_dtype, int64_t row_stride, int64_t seq_stride,
                             const float *row_max, const float *row_sum,
                             const float *q_rows, const int32_t *draft_ids,
                             const int32_t *tgt_ids, const float *q_prime,
                             const int32_t *span_start, const int32_t *span_len,
                             const int32_t *m, const uint8_t *tail_kind,
                             const int32_t *n_accepted, const float *temperature,
                             const uint64_t *seed, uint64_t step, int32_t *out_token,
                             float *resid_mass, uint32_t *sample_flags, void *stream);

/* ---- misc ---------------------------------------------------------------- */

/* Launch shape of the last od_verify / od_sample_residual call on this context
 * (for benchmarks). which: 0 = verify grid size, 1 = 512-byte units of row 0 data per
 * thread block, 2 = sample grid size, 3 = sample tiles per warp. */
int64_t od_last_launch_info(const od_ctx *ctx, int32_t which);

const char *od_status_string(int32_t status);
int32_t od_version(void);

#ifdef __cplusplus
}
#endif
#endif /* OMNIDRAFT_H */
