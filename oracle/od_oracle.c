/*
 * CPU oracle for the cross-vocabulary speculative-verification step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the step computes, written from the paper; the CUDA library is checked
 * against it.  It shares no code, header, table or helper with the CUDA
 * path, and nothing on the product path may call it.
 *
 * What it follows (OmniDraft, arXiv 2507.02659):
 *   - Section 3.1, Eq. (1): translation of a draft proposal d_t..d_{t+k-1}
 *     into m target tokens t_i with draft probabilities q'(t_i): a token
 *     with a direct map keeps q(d_i); a run of sub-tokens that hits the
 *     n-gram cache becomes one target token with q' = prod_j q(d_j).
 *   - Section 3.1, Eq. (2): the full mapped distribution q'(.) over the
 *     target vocabulary used by the correction step.
 *   - Notation paragraph of Section 3: residual norm(max(0, p - q)).
 *   - Algorithm 1, the translation / verification / free-token lines:
 *     acceptance ratio min(1, p(t_i)/q'(t_i)), accepted prefix length n,
 *     residual sample at the first rejection, free token when n == m.
 *
 * All floating point is fp64; sums run in index order; nothing is blocked,
 * fused or reordered.
 *
 * Readings taken where the paper is silent (each also listed in the design
 * notes of the repository):
 *   R1  merge scan is greedy left to right, longest cached run first (4..2)
 *   R2  the cache is tried before the direct map at every offset (the
 *       examples table of App. D merges two directly mapped tokens)
 *   R3  cached runs have 2..4 draft tokens
 *   R4  a run cut off by the end of the proposal does not match
 *   R5  a draft token with neither a cache hit nor a direct map ends the
 *       proposal: forced rejection at that position, the extra token is
 *       drawn from norm(max(0, p - q')) with the sub-normalised q'
 *   R7  "q(t) otherwise" in Eq. (2) is the drafter's row at the first
 *       sub-token of the run
 *   R8  Eq. (2) cases apply in the order written
 *   R9  Eq. (2) adjusts only for the n-gram at the rejected position
 *   R10 accept iff u < ratio with u in [0,1) on a 24-bit grid
 *   R12 inverse CDF in target-id order, strict '>'
 *
 * Pins (tests/test_oracle_*.py): lossless Monte-Carlo invariant, closed-form
 * acceptance sum_t min(p,q'), brute-force segmentation, hand example of
 * Eq. (2) with mass conservation, library softmax, Philox known answers.
 * Parity unpinned (nothing in the paper fixes them): the 24-bit uniform
 * construction and the counter layout (step, position, tag) of the random
 * stream.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OD_ORACLE_NMAX 4

enum { ORACLE_TAIL_COMPLETE = 0, ORACLE_TAIL_UNMAPPED_STOP = 1 };
enum { ORACLE_KIND_RESIDUAL = 0, ORACLE_KIND_BONUS = 1 };
enum { ORACLE_FLAG_ZERO_MASS = 1, ORACLE_FLAG_BAD_TEMPERATURE = 2 };

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
 * as easy as 1, 2, 3", SC'11).  Counter-based: 128-bit counter, 64-bit
 * key, ten rounds, key bumped by the Weyl constants between rounds.   */

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2],
                          uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* One uniform per (sequence seed, step, position, purpose): key = seed,
 * counter = (step lo, step hi, position, tag); the top 24 bits of the
 * first output word, scaled by 2^-24: exact in fp32 and fp64, in [0,1). */
double oracle_uniform(uint64_t seed, uint64_t step, uint32_t position,
                      uint32_t tag)
{
    uint32_t ctr[4] = { (uint32_t)step, (uint32_t)(step >> 32), position, tag };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t w[4];
    oracle_philox4x32_10(ctr, key, w);
    return (double)(w[0] >> 8) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------------ */
/* n-gram cache C = {(t, [d_1..d_n])} (Section 3.1): an exact-match
 * dictionary from a run of draft ids to one target id.  Held as an array
 * sorted by (length, ids); the first entry given for a run wins, as
 * Algorithm 1 only adds an n-gram that is not in the cache yet.        */

typedef struct {
    int32_t ids[OD_ORACLE_NMAX];
    int32_t len;
    int32_t target;
    int64_t order;
} oracle_entry;

typedef struct {
    oracle_entry *e;
    int64_t n;
} oracle_cache;

static int entry_key_cmp(const oracle_entry *a, const oracle_entry *b)
{
    if (a->len != b->len) return a->len < b->len ? -1 : 1;
    for (int j = 0; j < a->len; ++j)
        if (a->ids[j] != b->ids[j]) return a->ids[j] < b->ids[j] ? -1 : 1;
    return 0;
}

static int entry_sort_cmp(const void *pa, const void *pb)
{
    const oracle_entry *a = (const oracle_entry *)pa;
    const oracle_entry *b = (const oracle_entry *)pb;
    int c = entry_key_cmp(a, b);
    if (c) return c;
    return a->order < b->order ? -1 : (a->order > b->order ? 1 : 0);
}

static int entry_find_cmp(const void *pa, const void *pb)
{
    return entry_key_cmp((const oracle_entry *)pa, (const oracle_entry *)pb);
}

/* runs: [E][4] (unused = -1), len: [E] in 2..4, target: [E].  Returns NULL
 * on a malformed entry. */
oracle_cache *oracle_cache_create(const int32_t *runs, const int32_t *len,
                                  const int32_t *target, int64_t E)
{
    oracle_cache *c = (oracle_cache *)calloc(1, sizeof(*c));
    if (!c) return NULL;
    c->e = (oracle_entry *)calloc((size_t)(E > 0 ? E : 1), sizeof(oracle_entry));
    if (!c->e) { free(c); return NULL; }
    for (int64_t i = 0; i < E; ++i) {
        if (len[i] < 2 || len[i] > OD_ORACLE_NMAX) { free(c->e); free(c); return NULL; }
        for (int j = 0; j < OD_ORACLE_NMAX; ++j)
            c->e[i].ids[j] = j < len[i] ? runs[i * OD_ORACLE_NMAX + j] : -1;
        c->e[i].len = len[i];
        c->e[i].target = target[i];
        c->e[i].order = i;
    }
    qsort(c->e, (size_t)E, sizeof(oracle_entry), entry_sort_cmp);
    int64_t w = 0;
    for (int64_t i = 0; i < E; ++i)
        if (w == 0 || entry_key_cmp(&c->e[w - 1], &c->e[i]) != 0) c->e[w++] = c->e[i];
    c->n = w;
    return c;
}

void oracle_cache_destroy(oracle_cache *c)
{
    if (c) { free(c->e); free(c); }
}

int64_t oracle_cache_size(const oracle_cache *c) { return c ? c->n : 0; }

/* lookup([d_1..d_len], C): the target id, or -1 on a miss. */
int32_t oracle_cache_lookup(const oracle_cache *c, const int32_t *ids, int32_t len)
{
    if (!c || c->n == 0 || len < 2 || len > OD_ORACLE_NMAX) return -1;
    oracle_entry k;
    memset(&k, 0, sizeof(k));
    for (int j = 0; j < len; ++j) k.ids[j] = ids[j];
    k.len = len;
    const oracle_entry *hit = (const oracle_entry *)bsearch(
        &k, c->e, (size_t)c->n, sizeof(oracle_entry), entry_find_cmp);
    return hit ? hit->target : -1;
}

/* ------------------------------------------------------------------ */
/* Eq. (1): translate one proposal.  Outputs hold K entries (span_start has
 * one more meaning: span_start[m] is the position of the stopping token
 * under UNMAPPED_STOP).  Returns the number of cache hits.             */

int32_t oracle_map_sequence(const oracle_cache *cache, const int32_t *vocab_map,
                            int32_t V_q, const int32_t *d, int32_t K,
                            const float *q_sel, int32_t *tgt, double *q_prime,
                            int32_t *span_start, int32_t *span_len,
                            int32_t *m_out, int32_t *tail_kind)
{
    int32_t s = 0, m = 0, hits = 0;
    *tail_kind = ORACLE_TAIL_COMPLETE;
    while (s < K) {
        int32_t matched = 0;
        /* a run may only use ids of the draft vocabulary */
        for (int32_t L = OD_ORACLE_NMAX; L >= 2 && !matched; --L) {
            if (s + L > K) continue;                       /* R4 */
            int ok = 1;
            for (int32_t j = 0; j < L; ++j)
                if (d[s + j] < 0 || d[s + j] >= V_q) ok = 0;
            if (!ok) continue;
            int32_t t = oracle_cache_lookup(cache, d + s, L);
            if (t >= 0) {
                double prod = 1.0;
                for (int32_t j = 0; j < L; ++j) prod *= (double)q_sel[s + j];
                tgt[m] = t; q_prime[m] = prod;
                span_start[m] = s; span_len[m] = L;
                ++m; s += L; ++hits; matched = 1;
            }
        }
        if (matched) continue;
        int32_t direct = (d[s] >= 0 && d[s] < V_q) ? vocab_map[d[s]] : -1;
        if (direct >= 0) {
            tgt[m] = direct; q_prime[m] = (double)q_sel[s];
            span_start[m] = s; span_len[m] = 1;
            ++m; ++s;
        } else {                                           /* R5 */
            span_start[m] = s; span_len[m] = 1;
            *tail_kind = ORACLE_TAIL_UNMAPPED_STOP;
            break;
        }
    }
    *m_out = m;
    return hits;
}

/* ------------------------------------------------------------------ */
/* target logits are fp32 (dtype 0) or bf16 (dtype 1); both widen exactly. */

static double logit_at(const void *base, int32_t dtype, int64_t idx)
{
    if (dtype == 0) return (double)((const float *)base)[idx];
    uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
    float f;
    memcpy(&f, &bits, sizeof(f));
    return (double)f;
}

/* p(.) = softmax(x / T) over one row: M = max x, S = sum exp((x - M)/T). */
void oracle_row_stats(const void *row, int32_t dtype, int64_t V, double T,
                      double *M_out, double *S_out)
{
    double M = -INFINITY;
    for (int64_t t = 0; t < V; ++t) {
        double x = logit_at(row, dtype, t);
        if (x > M) M = x;
    }
    double S = 0.0;
    for (int64_t t = 0; t < V; ++t)
        S += exp((logit_at(row, dtype, t) - M) / T);
    *M_out = M; *S_out = S;
}

/* writes p(t) for every t of one row */
void oracle_softmax_row(const void *row, int32_t dtype, int64_t V, double T,
                        double *p)
{
    double M, S;
    oracle_row_stats(row, dtype, V, T, &M, &S);
    for (int64_t t = 0; t < V; ++t)
        p[t] = exp((logit_at(row, dtype, t) - M) / T) / S;
}

/* Eq. (2): q'(.) over the target vocabulary for the proposal position whose
 * run starts at draft position `start` with `len` sub-tokens.  `q_row` is the
 * drafter's distribution at `start`; ngram_token/ngram_prob describe the
 * cached n-gram at this position (len >= 2), ignored when len == 1.     */
void oracle_full_mapping(const float *q_row, int32_t V_q, const int32_t *vocab_map,
                         int64_t V_p, int32_t first_draft_id, int32_t len,
                         int32_t ngram_token, double ngram_prob, double *q_full)
{
    for (int64_t t = 0; t < V_p; ++t) q_full[t] = 0.0;
    for (int32_t dd = 0; dd < V_q; ++dd)                 /* q(t) otherwise */
        if (vocab_map[dd] >= 0) q_full[vocab_map[dd]] = (double)q_row[dd];
    if (len >= 2) {
        int32_t pre = (first_draft_id >= 0 && first_draft_id < V_q)
                          ? vocab_map[first_draft_id] : -1;
        if (pre >= 0)                                    /* prefix sub-token */
            q_full[pre] = (double)q_row[first_draft_id] - ngram_prob;
        q_full[ngram_token] = ngram_prob;                /* n-gram mapped */
    }
}

/* Inverse-CDF draw from r(.) / sum r: smallest t with C_t > u * R (R12).
 * Also reports the CDF interval [C_{probe-1}, C_probe] of `probe` (pass -1
 * to skip).  Returns the token, or -1 when R <= 0.                      */
static int64_t inverse_cdf(const double *r, int64_t V, double u, double *R_out,
                           int64_t probe, double *probe_lo, double *probe_hi)
{
    double R = 0.0;
    for (int64_t t = 0; t < V; ++t) R += r[t];
    *R_out = R;
    if (!(R > 0.0)) return -1;
    double target = u * R, C = 0.0;
    int64_t pick = -1, last_pos = -1;
    for (int64_t t = 0; t < V; ++t) {
        double lo = C;
        C += r[t];
        if (t == probe) { *probe_lo = lo; *probe_hi = C; }
        if (r[t] > 0.0) last_pos = t;
        if (pick < 0 && C > target) pick = t;
    }
    return pick >= 0 ? pick : last_pos;
}

/* ------------------------------------------------------------------ */
/* One verification step for one sequence (Algorithm 1, translation through
 * free token).  Arrays indexed by proposal position hold K_max entries.  */

void oracle_step_sequence(const oracle_cache *cache, const int32_t *vocab_map,
                          int32_t V_q, int64_t V_p, int32_t K_max,
                          const int32_t *draft_ids, int32_t K,
                          const float *q_sel, const float *q_rows,
                          const void *logits, int32_t logit_dtype,
                          int64_t row_stride, double T, uint64_t seed,
                          uint64_t step, int32_t probe_token,
                          /* outputs */
                          int32_t *tgt, double *q_prime, int32_t *span_start,
                          int32_t *span_len, int32_t *m_out, int32_t *tail_out,
                          int32_t *hits_out, double *row_max, double *row_sum,
                          double *p_sel, double *ratio, double *u_acc,
                          int32_t *accept, int32_t *n_out, int32_t *n_draft_out,
                          int32_t *kind_out, int32_t *token_out, double *mass_out,
                          double *u_samp_out, double *cdf_lo, double *cdf_hi,
                          double *probe_lo, double *probe_hi, int32_t *flags_out)
{
    int32_t m = 0, tail = 0, flags = 0;
    if (K < 0) K = 0;
    if (K > K_max) K = K_max;
    *hits_out = oracle_map_sequence(cache, vocab_map, V_q, draft_ids, K, q_sel,
                                    tgt, q_prime, span_start, span_len, &m, &tail);
    *m_out = m; *tail_out = tail;
    *probe_lo = *probe_hi = *cdf_lo = *cdf_hi = *mass_out = *u_samp_out = 0.0;
    *token_out = -1; *kind_out = 0; *n_out = 0; *n_draft_out = 0;
    if (!(T > 0.0)) {             /* greedy decoding is not part of this path */
        *flags_out = ORACLE_FLAG_BAD_TEMPERATURE;
        return;
    }

    size_t esz = logit_dtype == 0 ? 4 : 2;
    for (int32_t r = 0; r <= m; ++r)
        oracle_row_stats((const char *)logits + (size_t)r * row_stride * esz,
                         logit_dtype, V_p, T, &row_max[r], &row_sum[r]);

    /* acceptance test at every proposed position, prefix = leading accepts */
    int32_t n = m;
    for (int32_t i = 0; i < m; ++i) {
        const char *row = (const char *)logits + (size_t)i * row_stride * esz;
        double x = logit_at(row, logit_dtype, tgt[i]);
        p_sel[i] = exp((x - row_max[i]) / T) / row_sum[i];
        ratio[i] = (q_prime[i] <= p_sel[i]) ? 1.0 : p_sel[i] / q_prime[i];
        u_acc[i] = oracle_uniform(seed, step, (uint32_t)i, 0u);
        accept[i] = u_acc[i] < ratio[i];
        if (!accept[i] && n == m) n = i;
    }
    *n_out = n;
    int32_t nd = 0;
    for (int32_t i = 0; i < n; ++i) nd += span_len[i];
    *n_draft_out = nd;

    /* the extra token at position j = n */
    int32_t j = n;
    const char *row = (const char *)logits + (size_t)j * row_stride * esz;
    double *p = (double *)malloc(sizeof(double) * (size_t)V_p);
    double *r = (double *)malloc(sizeof(double) * (size_t)V_p);
    oracle_softmax_row(row, logit_dtype, V_p, T, p);
    int32_t kind;
    if (j < m || tail == ORACLE_TAIL_UNMAPPED_STOP) {
        kind = ORACLE_KIND_RESIDUAL;
        int32_t s0 = span_start[j];
        int32_t len = j < m ? span_len[j] : 1;
        oracle_full_mapping(q_rows + (size_t)s0 * V_q, V_q, vocab_map, V_p,
                            draft_ids[s0], len, j < m ? tgt[j] : -1,
                            j < m ? q_prime[j] : 0.0, r);
        for (int64_t t = 0; t < V_p; ++t) {
            double diff = p[t] - r[t];
            r[t] = diff > 0.0 ? diff : 0.0;
        }
    } else {
        kind = ORACLE_KIND_BONUS;
        for (int64_t t = 0; t < V_p; ++t) r[t] = p[t];
    }
    double u = oracle_uniform(seed, step, (uint32_t)j, 1u);
    double R = 0.0;
    int64_t tok = inverse_cdf(r, V_p, u, &R, probe_token, probe_lo, probe_hi);
    if (tok < 0) {               /* no residual mass: fall back to p_j */
        flags |= ORACLE_FLAG_ZERO_MASS;
        tok = inverse_cdf(p, V_p, u, &R, probe_token, probe_lo, probe_hi);
        memcpy(r, p, sizeof(double) * (size_t)V_p);
    }
    double C = 0.0;
    for (int64_t t = 0; t < tok; ++t) C += r[t];
    *cdf_lo = C; *cdf_hi = C + r[tok];
    *kind_out = kind; *token_out = (int32_t)tok; *mass_out = R; *u_samp_out = u;
    *flags_out = flags;
    free(p); free(r);
}

/* A batch of independent sequences; `threads` > 1 splits them over OpenMP
 * threads (the only parallelism in this file).  Layouts, K = K_max:
 *   draft_ids i32[B,K]  draft_len i32[B]  q_sel f32[B,K]  q_rows f32[B,K,V_q]
 *   logits [B,K+1,V_p] with the given row / sequence strides in elements
 *   per-position outputs [B,K]; row_max/row_sum [B,K+1]; per-sequence [B]. */
void oracle_step_batch(const oracle_cache *cache, const int32_t *vocab_map,
                       int32_t V_q, int64_t V_p, int32_t B, int32_t K_max,
                       const int32_t *draft_ids, const int32_t *draft_len,
                       const float *q_sel, const float *q_rows,
                       const void *logits, int32_t logit_dtype,
                       int64_t row_stride, int64_t seq_stride,
                       const float *temperature, const uint64_t *seed,
                       uint64_t step, const int32_t *probe_token, int32_t threads,
                       int32_t *tgt, double *q_prime, int32_t *span_start,
                       int32_t *span_len, int32_t *m, int32_t *tail,
                       int32_t *hits, double *row_max, double *row_sum,
                       double *p_sel, double *ratio, double *u_acc,
                       int32_t *accept, int32_t *n_acc, int32_t *n_draft,
                       int32_t *kind, int32_t *token, double *mass,
                       double *u_samp, double *cdf_lo, double *cdf_hi,
                       double *probe_lo, double *probe_hi, int32_t *flags)
{
    size_t esz = logit_dtype == 0 ? 4 : 2;
    int32_t K = K_max;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 0 ? threads : 1)
#endif
    for (int32_t b = 0; b < B; ++b) {
        size_t o = (size_t)b * K;
        oracle_step_sequence(
            cache, vocab_map, V_q, V_p, K_max, draft_ids + o, draft_len[b],
            q_sel + o, q_rows + o * (size_t)V_q,
            (const char *)logits + (size_t)b * seq_stride * esz, logit_dtype,
            row_stride, (double)temperature[b], seed[b], step,
            probe_token ? probe_token[b] : -1,
            tgt + o, q_prime + o, span_start + o, span_len + o, m + b, tail + b,
            hits + b, row_max + (size_t)b * (K + 1), row_sum + (size_t)b * (K + 1),
            p_sel + o, ratio + o, u_acc + o, accept + o, n_acc + b, n_draft + b,
            kind + b, token + b, mass + b, u_samp + b, cdf_lo + b, cdf_hi + b,
            probe_lo + b, probe_hi + b, flags + b);
    }
}

int32_t oracle_openmp_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
