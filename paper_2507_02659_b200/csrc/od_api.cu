// C ABI of the library (see include/omnidraft.h): context life cycle, the
// host-side builds of the vocabulary map and of the n-gram cache table,
// argument validation, and the whole-step entry point for host buffers.
#include <algorithm>
#include <new>
#include <string.h>
#include <vector>

#include "od_common.cuh"

namespace {

#define OD_CUDA(call)                                  \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) return OD_ERR_CUDA;    \
    } while (0)

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

template <typename T>
int32_t dev_alloc(T **p, size_t n)
{
    *p = nullptr;
    if (n == 0) n = 1;
    cudaError_t e = cudaMalloc((void **)p, n * sizeof(T));
    if (e == cudaErrorMemoryAllocation) return OD_ERR_NOMEM;
    if (e != cudaSuccess) return OD_ERR_CUDA;
    e = cudaMemset(*p, 0, n * sizeof(T));
    return e == cudaSuccess ? OD_OK : OD_ERR_CUDA;
}

void free_all(od_ctx *c)
{
    od_cache_free_dynamic(c);
    void *ptrs[] = {c->d_vocab_map, c->d_inv_map, c->d_keys, c->d_vals, c->d_partials,
                    c->d_tile_sums,
                    c->d_samp_ticket, c->s_logits, c->s_q_rows, c->s_q_sel, c->s_temperature,
                    c->s_draft_ids, c->s_draft_len, c->s_seed, c->s_tgt_ids, c->s_span_start,
                    c->s_span_len, c->s_m, c->s_n_acc, c->s_n_draft, c->s_token, c->s_q_prime,
                    c->s_row_max, c->s_row_sum, c->s_p_sel, c->s_ratio, c->s_mass, c->s_tail,
                    c->s_vflags, c->s_sflags};
    for (void *p : ptrs)
        if (p) cudaFree(p);
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

int32_t check_step_common(const od_ctx *c, int32_t B, int32_t K_max)
{
    if (!c) return OD_ERR_INVALID_ARG;
    if (B < 0 || B > c->max_batch) return OD_ERR_INVALID_ARG;
    if (K_max < 1 || K_max > c->max_k) return OD_ERR_INVALID_ARG;
    if (!c->have_map) return OD_ERR_STATE;
    return OD_OK;
}

// row_len: elements of a row (the whole vocabulary, or a shard's columns)
int32_t check_logits_len(int64_t row_len, const void *logits, int32_t dtype, int64_t row_stride,
                         int64_t seq_stride, int32_t K_max)
{
    if (!logits) return OD_ERR_INVALID_ARG;
    if (dtype != OD_F32 && dtype != OD_BF16) return OD_ERR_UNSUPPORTED;
    const int64_t esz = dtype == OD_BF16 ? 2 : 4;
    if (row_stride < row_len || seq_stride < row_stride * (K_max + 1)) return OD_ERR_INVALID_ARG;
    if (!aligned16(logits) || (row_stride * esz) % 16 != 0 || (seq_stride * esz) % 16 != 0)
        return OD_ERR_ALIGNMENT;
    return OD_OK;
}

int32_t check_logits(const od_ctx *c, const void *logits, int32_t dtype, int64_t row_stride,
                     int64_t seq_stride, int32_t K_max)
{
    return check_logits_len(c->v_p, logits, dtype, row_stride, seq_stride, K_max);
}

// a vocabulary shard: whole 256-id tiles, inside the vocabulary
int32_t check_shard(const od_ctx *c, int32_t shard_lo, int32_t shard_len)
{
    if (shard_lo < 0 || shard_len < 1 || (int64_t)shard_lo + shard_len > c->v_p) return OD_ERR_INVALID_ARG;
    if (shard_lo % OD_SAMPLE_TILE != 0) return OD_ERR_INVALID_ARG;
    const int32_t hi = shard_lo + shard_len;
    if (hi % OD_SAMPLE_TILE != 0 && hi != c->v_p) return OD_ERR_INVALID_ARG;
    return OD_OK;
}

}  // namespace

extern "C" {

int32_t od_create(od_ctx **ctx, int32_t device, int32_t draft_vocab, int32_t target_vocab,
                  int32_t max_batch, int32_t max_k)
{
    if (!ctx) return OD_ERR_INVALID_ARG;
    *ctx = nullptr;
    if (draft_vocab < 1 || target_vocab < 1 || max_batch < 1 || max_batch > 65535 ||
        max_k < 1 || max_k > OD_MAX_K)
        return OD_ERR_INVALID_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) return OD_ERR_CUDA;
    if (device < 0 || device >= ndev) return OD_ERR_INVALID_ARG;
    DeviceGuard g(device);
    if (!g.ok) return OD_ERR_CUDA;

    od_ctx *c = new (std::nothrow) od_ctx();
    if (!c) return OD_ERR_NOMEM;
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->v_q = draft_vocab; c->v_p = target_vocab; c->max_batch = max_batch; c->max_k = max_k;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        delete c;
        return OD_ERR_CUDA;
    }
    c->opt_pdl = 1;
    c->tiles_per_row = (target_vocab + OD_SAMPLE_TILE - 1) / OD_SAMPLE_TILE;
    // the sampler keeps a row's tile values in shared memory: that bounds the target vocabulary
    if (od_sample_smem_bytes(c->tiles_per_row) > OD_SAMPLE_SMEM_MAX) {
        delete c;
        return OD_ERR_UNSUPPORTED;
    }
    if (od_sample_prepare_device(od_sample_smem_bytes(c->tiles_per_row)) != cudaSuccess) {
        delete c;
        return OD_ERR_CUDA;
    }
    // od_verify scratch serves one launch: at most OD_VERIFY_MAX_B sequences
    const size_t vb = max_batch < OD_VERIFY_MAX_B ? max_batch : OD_VERIFY_MAX_B;
    const size_t rows = vb * (max_k + 1);
    int32_t st = OD_OK;
    if (st == OD_OK) st = dev_alloc(&c->d_vocab_map, (size_t)draft_vocab);
    if (st == OD_OK) st = dev_alloc(&c->d_inv_map, (size_t)target_vocab + 8);

    if (st == OD_OK) st = dev_alloc(&c->d_partials, rows * OD_VERIFY_SEG_MAX);
    if (st == OD_OK) st = dev_alloc(&c->d_tile_sums, (size_t)max_batch * c->tiles_per_row);
    if (st == OD_OK) st = dev_alloc(&c->d_samp_ticket, (size_t)max_batch);
    if (st != OD_OK) {
        free_all(c);
        delete c;
        return st;
    }
    *ctx = c;
    return OD_OK;
}

int32_t od_destroy(od_ctx *c)
{
    if (!c) return OD_OK;
    DeviceGuard g(c->device);
    if (g.ok) cudaDeviceSynchronize();
    free_all(c);
    delete c;
    return OD_OK;
}

int32_t od_set_vocab_map(od_ctx *c, const int32_t *host_map)
{
    if (!c || !host_map) return OD_ERR_INVALID_ARG;
    std::vector<int32_t> inv((size_t)c->v_p, -1);
    for (int32_t d = 0; d < c->v_q; ++d) {
        const int32_t t = host_map[d];
        if (t < 0) continue;
        if (t >= c->v_p) return OD_ERR_INVALID_ARG;
        if (inv[t] >= 0) return OD_ERR_MAP_NOT_INJECTIVE;
        inv[t] = d;
    }
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(cudaDeviceSynchronize());
    // store -1 for every unmapped id, whatever negative value the caller used
    std::vector<int32_t> fwd((size_t)c->v_q);
    for (int32_t d = 0; d < c->v_q; ++d) fwd[d] = host_map[d] < 0 ? -1 : host_map[d];
    OD_CUDA(cudaMemcpy(c->d_vocab_map, fwd.data(), fwd.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    OD_CUDA(cudaMemcpy(c->d_inv_map, inv.data(), inv.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    c->have_map = true;
    return OD_OK;
}

int32_t od_cache_build(od_ctx *c, const int32_t *host_runs, const int32_t *host_len,
                       const int32_t *host_target, int64_t E)
{
    if (!c || E < 0) return OD_ERR_INVALID_ARG;
    if (E > 0 && (!host_runs || !host_len || !host_target)) return OD_ERR_INVALID_ARG;
    if (E > 0 && c->v_q > 65535) return OD_ERR_UNSUPPORTED;
    if (E > ((int64_t)1 << 30)) return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;

    int64_t cap = 0;
    std::vector<uint64_t> keys;
    std::vector<int32_t> vals;
    if (E > 0) {
        cap = 64;
        while (cap < 2 * E) cap <<= 1;
        keys.assign((size_t)cap, 0ULL);
        vals.assign((size_t)cap, -1);
        const uint64_t ngroups = (uint64_t)cap / OD_GROUP;
        for (int64_t e = 0; e < E; ++e) {
            const int32_t L = host_len[e];
            if (L < 2 || L > OD_NGRAM_MAX) return OD_ERR_BAD_CACHE_ENTRY;
            const int32_t *ids = host_runs + e * OD_NGRAM_MAX;
            for (int j = 0; j < L; ++j)
                if (ids[j] < 0 || ids[j] >= c->v_q) return OD_ERR_BAD_CACHE_ENTRY;
            if (host_target[e] < 0 || host_target[e] >= c->v_p) return OD_ERR_BAD_CACHE_ENTRY;
            const uint64_t key = od_pack_run(ids, L);
            uint64_t grp = od_hash64(key) & (ngroups - 1);
            bool done = false;
            for (uint64_t step = 0; step < ngroups && !done; ++step) {
                uint64_t *gk = keys.data() + grp * OD_GROUP;
                for (int s = 0; s < OD_GROUP; ++s) {
                    if (gk[s] == key) { done = true; break; }          // first entry wins
                    if (gk[s] == 0ULL) {
                        gk[s] = key;
                        vals[grp * OD_GROUP + s] = host_target[e];
                        done = true;
                        break;
                    }
                }
                grp = (grp + 1) & (ngroups - 1);
            }
            if (!done) return OD_ERR_NOMEM;                            // cannot happen at load <= 1/2
        }
    }
    OD_CUDA(cudaDeviceSynchronize());
    od_cache_free_dynamic(c);                               // a static cache replaces an online one
    if (c->d_keys) { cudaFree(c->d_keys); c->d_keys = nullptr; }
    if (c->d_vals) { cudaFree(c->d_vals); c->d_vals = nullptr; }
    c->cap = 0;
    if (cap > 0) {
        int32_t st = dev_alloc(&c->d_keys, (size_t)cap);
        if (st == OD_OK) st = dev_alloc(&c->d_vals, (size_t)cap);
        if (st != OD_OK) return st;
        OD_CUDA(cudaMemcpy(c->d_keys, keys.data(), (size_t)cap * sizeof(uint64_t), cudaMemcpyHostToDevice));
        OD_CUDA(cudaMemcpy(c->d_vals, vals.data(), (size_t)cap * sizeof(int32_t), cudaMemcpyHostToDevice));
        c->cap = cap;
    }
    return OD_OK;
}

int32_t od_set_option(od_ctx *c, const char *name, int64_t value)
{
    if (!c || !name || value < 0) return OD_ERR_INVALID_ARG;
    if (!strcmp(name, "verify_grid")) { c->opt_verify_grid = value; return OD_OK; }
    if (!strcmp(name, "early_inputs")) { c->opt_early_inputs = value != 0; return OD_OK; }
    if (!strcmp(name, "sample_tiles_per_warp")) { c->opt_sample_tiles_per_warp = value; return OD_OK; }
    if (!strcmp(name, "pdl")) { c->opt_pdl = value != 0; return OD_OK; }
    return OD_ERR_INVALID_ARG;
}

int32_t od_map_proposals(od_ctx *c, int32_t B, int32_t K_max, const int32_t *draft_ids,
                         const int32_t *draft_len, const float *q_sel, int32_t *tgt_ids,
                         float *q_prime, int32_t *span_start, int32_t *span_len, int32_t *m,
                         uint8_t *tail_kind, uint32_t *counters, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    if (!draft_ids || !draft_len || !q_sel || !tgt_ids || !q_prime || !span_start || !span_len ||
        !m || !tail_kind)
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(od_launch_map(c, B, K_max, draft_ids, draft_len, q_sel, tgt_ids, q_prime, span_start,
                          span_len, m, tail_kind, counters, c->opt_early_inputs != 0, false, (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_verify(od_ctx *c, int32_t B, int32_t K_max, const void *logits, int32_t logit_dtype,
                  int64_t row_stride, int64_t seq_stride, const int32_t *tgt_ids,
                  const float *q_prime, const int32_t *span_len, const int32_t *m,
                  const float *temperature, const uint64_t *seed, uint64_t step, float *row_max,
                  float *row_sum, float *p_sel, float *ratio, int32_t *n_accepted,
                  int32_t *n_draft_accepted, uint32_t *verify_flags, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    st = check_logits(c, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!tgt_ids || !q_prime || !span_len || !m || !temperature || !seed || !row_max || !row_sum ||
        !p_sel || !ratio || !n_accepted || !n_draft_accepted || !verify_flags)
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    c->verify_early = c->opt_early_inputs != 0;
    OD_CUDA(od_launch_verify(c, B, K_max, logits, logit_dtype, row_stride, seq_stride, tgt_ids,
                             q_prime, span_len, m, temperature, seed, step, row_max, row_sum,
                             p_sel, ratio, n_accepted, n_draft_accepted, verify_flags,
                             (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_sample_residual(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                           int32_t logit_dtype, int64_t row_stride, int64_t seq_stride,
                           const float *row_max, const float *row_sum, const float *q_rows,
                           const int32_t *draft_ids, const int32_t *tgt_ids, const float *q_prime,
                           const int32_t *span_start, const int32_t *span_len, const int32_t *m,
                           const uint8_t *tail_kind, const int32_t *n_accepted,
                           const float *temperature, const uint64_t *seed, uint64_t step,
                           int32_t *out_token, float *resid_mass, uint32_t *sample_flags,
                           void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    st = check_logits(c, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!row_max || !row_sum || !q_rows || !draft_ids || !tgt_ids || !q_prime || !span_start ||
        !span_len || !m || !tail_kind || !n_accepted || !temperature || !seed || !out_token ||
        !resid_mass || !sample_flags)
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(od_launch_sample(c, B, K_max, logits, logit_dtype, row_stride, seq_stride, row_max,
                             row_sum, q_rows, draft_ids, tgt_ids, q_prime, span_start, span_len, m,
                             tail_kind, n_accepted, temperature, seed, step, out_token, resid_mass,
                             sample_flags, (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_step(od_ctx *c, int32_t B, int32_t K_max, const int32_t *draft_ids, const int32_t *draft_len,
                const float *q_sel, const float *q_rows, const void *logits, int32_t logit_dtype,
                int64_t row_stride, int64_t seq_stride, const float *temperature, const uint64_t *seed,
                uint64_t step, int32_t *tgt_ids, float *q_prime, int32_t *span_start, int32_t *span_len,
                int32_t *m, uint8_t *tail_kind, uint32_t *counters, float *row_max, float *row_sum,
                float *p_sel, float *ratio, int32_t *n_accepted, int32_t *n_draft_accepted,
                uint32_t *verify_flags, int32_t *out_token, float *resid_mass, uint32_t *sample_flags,
                void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    st = check_logits(c, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!draft_ids || !draft_len || !q_sel || !q_rows || !temperature || !seed || !tgt_ids || !q_prime ||
        !span_start || !span_len || !m || !tail_kind || !row_max || !row_sum || !p_sel || !ratio ||
        !n_accepted || !n_draft_accepted || !verify_flags || !out_token || !resid_mass || !sample_flags)
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    OD_CUDA(od_launch_map(c, B, K_max, draft_ids, draft_len, q_sel, tgt_ids, q_prime, span_start, span_len, m,
                          tail_kind, counters, c->opt_early_inputs != 0, c->opt_early_inputs != 0, s));
    // The translation kernel waits for everything in front of it before it lets the next
    // kernel start, so whatever wrote the logits has finished by the time a block of the
    // stream kernel runs: rows 0 may be read before that kernel's own wait.
    c->verify_early = true;
    if (B > 0 && B <= od_verify_slice(K_max, c->v_p, logit_dtype) && c->opt_pdl) {
        // Three launches, not four: the streaming pass, then the sampler, whose blocks merge the
        // pass's partials and take step 2's decisions themselves (identical arithmetic) instead
        // of waiting for a decide kernel in between.
        od_fused_verify fuse = {};
        fuse.row_max = row_max; fuse.row_sum = row_sum; fuse.p_sel = p_sel; fuse.ratio = ratio;
        fuse.n_accepted = n_accepted; fuse.n_draft_accepted = n_draft_accepted; fuse.flags = verify_flags;
        OD_CUDA(od_launch_verify_stream(c, B, K_max, logits, logit_dtype, row_stride, seq_stride, m, temperature,
                                        &fuse, s));
        OD_CUDA(od_launch_sample(c, B, K_max, logits, logit_dtype, row_stride, seq_stride, row_max, row_sum,
                                 q_rows, draft_ids, tgt_ids, q_prime, span_start, span_len, m, tail_kind,
                                 n_accepted, temperature, seed, step, out_token, resid_mass, sample_flags, s,
                                 &fuse));
        return OD_OK;
    }
    OD_CUDA(od_launch_verify(c, B, K_max, logits, logit_dtype, row_stride, seq_stride, tgt_ids, q_prime,
                             span_len, m, temperature, seed, step, row_max, row_sum, p_sel, ratio,
                             n_accepted, n_draft_accepted, verify_flags, s));
    OD_CUDA(od_launch_sample(c, B, K_max, logits, logit_dtype, row_stride, seq_stride, row_max, row_sum,
                             q_rows, draft_ids, tgt_ids, q_prime, span_start, span_len, m, tail_kind,
                             n_accepted, temperature, seed, step, out_token, resid_mass, sample_flags, s));
    return OD_OK;
}

int32_t od_verify_shard_stats(od_ctx *c, int32_t B, int32_t K_max, int32_t shard_lo, int32_t shard_len,
                              const void *logits, int32_t logit_dtype, int64_t row_stride,
                              int64_t seq_stride, const int32_t *tgt_ids, const int32_t *m,
                              const float *temperature, float *stats, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    st = check_shard(c, shard_lo, shard_len);
    if (st != OD_OK) return st;
    st = check_logits_len(shard_len, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!tgt_ids || !m || !temperature || !stats) return OD_ERR_INVALID_ARG;
    if (!aligned16(stats)) return OD_ERR_ALIGNMENT;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    c->verify_early = c->opt_early_inputs != 0;
    OD_CUDA(od_launch_verify_shard_stats(c, B, K_max, shard_lo, shard_len, logits, logit_dtype, row_stride,
                                         seq_stride, tgt_ids, m, temperature, stats, (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_verify_shard_finish(od_ctx *c, int32_t B, int32_t K_max, int32_t n_shards,
                               const float *stats_all, const int32_t *tgt_ids, const float *q_prime,
                               const int32_t *span_len, const int32_t *m, const float *temperature,
                               const uint64_t *seed, uint64_t step, float *row_max, float *row_sum,
                               float *p_sel, float *ratio, int32_t *n_accepted,
                               int32_t *n_draft_accepted, uint32_t *verify_flags, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    if (n_shards < 1 || n_shards > 1024) return OD_ERR_INVALID_ARG;
    if (!stats_all || !tgt_ids || !q_prime || !span_len || !m || !temperature || !seed || !row_max ||
        !row_sum || !p_sel || !ratio || !n_accepted || !n_draft_accepted || !verify_flags)
        return OD_ERR_INVALID_ARG;
    if (!aligned16(stats_all)) return OD_ERR_ALIGNMENT;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(od_launch_verify_shard_finish(c, B, K_max, n_shards, stats_all, tgt_ids, q_prime, span_len, m,
                                          temperature, seed, step, row_max, row_sum, p_sel, ratio,
                                          n_accepted, n_draft_accepted, verify_flags, (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_sample_shard_mass(od_ctx *c, int32_t B, int32_t K_max, int32_t shard_lo, int32_t shard_len,
                             const void *logits, int32_t logit_dtype, int64_t row_stride,
                             int64_t seq_stride, const float *row_max, const float *row_sum,
                             const float *q_rows, const int32_t *draft_ids, const int32_t *tgt_ids,
                             const float *q_prime, const int32_t *span_start, const int32_t *span_len,
                             const int32_t *m, const uint8_t *tail_kind, const int32_t *n_accepted,
                             const float *temperature, double *mass, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    st = check_shard(c, shard_lo, shard_len);
    if (st != OD_OK) return st;
    st = check_logits_len(shard_len, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!row_max || !row_sum || !q_rows || !draft_ids || !tgt_ids || !q_prime || !span_start ||
        !span_len || !m || !tail_kind || !n_accepted || !temperature || !mass)
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(od_launch_sample_shard_mass(c, B, K_max, shard_lo, shard_len, logits, logit_dtype, row_stride,
                                        seq_stride, row_max, row_sum, q_rows, draft_ids, tgt_ids, q_prime,
                                        span_start, span_len, m, tail_kind, n_accepted, temperature, mass,
                                        (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_sample_shard_pick(od_ctx *c, int32_t B, int32_t K_max, int32_t n_shards, int32_t shard_index,
                             int32_t shard_lo, int32_t shard_len, const double *mass_all,
                             const void *logits, int32_t logit_dtype, int64_t row_stride,
                             int64_t seq_stride, const float *row_max, const float *row_sum,
                             const float *q_rows, const int32_t *draft_ids, const int32_t *tgt_ids,
                             const float *q_prime, const int32_t *span_start, const int32_t *span_len,
                             const int32_t *m, const uint8_t *tail_kind, const int32_t *n_accepted,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             int32_t *out_token, float *resid_mass, uint32_t *sample_flags, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    if (n_shards < 1 || n_shards > 1024 || shard_index < 0 || shard_index >= n_shards)
        return OD_ERR_INVALID_ARG;
    st = check_shard(c, shard_lo, shard_len);
    if (st != OD_OK) return st;
    st = check_logits_len(shard_len, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!mass_all || !row_max || !row_sum || !q_rows || !draft_ids || !tgt_ids || !q_prime ||
        !span_start || !span_len || !m || !tail_kind || !n_accepted || !temperature || !seed ||
        !out_token || !resid_mass || !sample_flags)
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(od_launch_sample_shard_pick(c, B, K_max, n_shards, shard_index, shard_lo, shard_len, mass_all,
                                        logits, logit_dtype, row_stride, seq_stride, row_max, row_sum,
                                        q_rows, draft_ids, tgt_ids, q_prime, span_start, span_len, m,
                                        tail_kind, n_accepted, temperature, seed, step, out_token,
                                        resid_mass, sample_flags, (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_distill_loss(od_ctx *c, int32_t B, int32_t K_max, const float *q_rows,
                        const int32_t *draft_ids, const int32_t *tgt_ids, const int32_t *span_start,
                        const int32_t *span_len, const int32_t *m, const void *logits,
                        int32_t logit_dtype, int64_t row_stride, int64_t seq_stride,
                        const float *row_max, const float *row_sum, const float *p_sel,
                        const float *temperature, float lambda, int32_t lambda_mode, float *loss,
                        float *grad, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    st = check_logits(c, logits, logit_dtype, row_stride, seq_stride, K_max);
    if (st != OD_OK) return st;
    if (!q_rows || !draft_ids || !tgt_ids || !span_start || !span_len || !m || !row_max || !row_sum ||
        !temperature || !loss || (lambda_mode != 0 && lambda_mode != 1) || (lambda_mode == 1 && !p_sel) ||
        !(lambda >= 0.f))
        return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    c->last_was_map = false;
    OD_CUDA(od_launch_distill(c, B, K_max, q_rows, draft_ids, tgt_ids, span_start, span_len, m, logits,
                              logit_dtype, row_stride, seq_stride, row_max, row_sum, p_sel, temperature,
                              lambda, lambda_mode, loss, grad, (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_exit_rule(od_ctx *c, int32_t B, int32_t K_max, const float *head_logits,
                     const int32_t *avail_len, float gamma, int32_t *draft_len, float *reject_prob,
                     uint32_t *exit_flags, void *stream)
{
    if (!c || B < 0 || K_max < 1 || K_max > OD_MAX_K) return OD_ERR_INVALID_ARG;
    if (!head_logits || !draft_len) return OD_ERR_INVALID_ARG;
    if (!(gamma >= 0.f && gamma <= 1.f)) return OD_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    c->last_was_map = false;
    OD_CUDA(od_launch_exit(B, K_max, head_logits, avail_len, gamma, draft_len, reject_prob, exit_flags,
                           (cudaStream_t)stream));
    return OD_OK;
}

int32_t od_host_step_reserve(od_ctx *c, int32_t logit_dtype)
{
    if (!c) return OD_ERR_INVALID_ARG;
    if (logit_dtype != OD_F32 && logit_dtype != OD_BF16) return OD_ERR_UNSUPPORTED;
    if (c->host_reserved) return c->host_dtype == logit_dtype ? OD_OK : OD_ERR_STATE;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    const size_t B = c->max_batch, K = c->max_k;
    const size_t esz = logit_dtype == OD_BF16 ? 2 : 4;
    int32_t st = OD_OK;
    char *lg = nullptr;
    st = dev_alloc(&lg, B * (K + 1) * (size_t)c->v_p * esz);
    c->s_logits = lg;
    if (st == OD_OK) st = dev_alloc(&c->s_q_rows, B * K * (size_t)c->v_q);
    if (st == OD_OK) st = dev_alloc(&c->s_q_sel, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_temperature, B);
    if (st == OD_OK) st = dev_alloc(&c->s_draft_ids, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_draft_len, B);
    if (st == OD_OK) st = dev_alloc(&c->s_seed, B);
    if (st == OD_OK) st = dev_alloc(&c->s_tgt_ids, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_span_start, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_span_len, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_m, B);
    if (st == OD_OK) st = dev_alloc(&c->s_n_acc, B);
    if (st == OD_OK) st = dev_alloc(&c->s_n_draft, B);
    if (st == OD_OK) st = dev_alloc(&c->s_token, B);
    if (st == OD_OK) st = dev_alloc(&c->s_q_prime, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_row_max, B * (K + 1));
    if (st == OD_OK) st = dev_alloc(&c->s_row_sum, B * (K + 1));
    if (st == OD_OK) st = dev_alloc(&c->s_p_sel, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_ratio, B * K);
    if (st == OD_OK) st = dev_alloc(&c->s_mass, B);
    if (st == OD_OK) st = dev_alloc(&c->s_tail, B);
    if (st == OD_OK) st = dev_alloc(&c->s_vflags, B);
    if (st == OD_OK) st = dev_alloc(&c->s_sflags, B);
    if (st != OD_OK) return st;
    c->host_reserved = true;
    c->host_dtype = logit_dtype;
    return OD_OK;
}

int32_t od_step_host(od_ctx *c, int32_t B, int32_t K_max, const int32_t *draft_ids,
                     const int32_t *draft_len, const float *q_sel, const float *q_rows,
                     const void *logits, int32_t logit_dtype, const float *temperature,
                     const uint64_t *seed, uint64_t step, int32_t *n_accepted,
                     int32_t *n_draft_accepted, int32_t *out_token, int32_t *tgt_ids, int32_t *m,
                     uint32_t *verify_flags, uint32_t *sample_flags, void *stream)
{
    int32_t st = check_step_common(c, B, K_max);
    if (st != OD_OK) return st;
    if (!c->host_reserved || c->host_dtype != logit_dtype) return OD_ERR_STATE;
    if (!draft_ids || !draft_len || !q_sel || !q_rows || !logits || !temperature || !seed)
        return OD_ERR_INVALID_ARG;
    if (B == 0) return OD_OK;
    DeviceGuard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t nB = B, K = K_max, esz = logit_dtype == OD_BF16 ? 2 : 4;
    const int64_t row_stride = c->v_p, seq_stride = (int64_t)c->v_p * (K_max + 1);
    if ((row_stride * (int64_t)esz) % 16 != 0) return OD_ERR_ALIGNMENT;
    const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;
    OD_CUDA(cudaMemcpyAsync(c->s_draft_ids, draft_ids, nB * K * 4, H2D, s));
    OD_CUDA(cudaMemcpyAsync(c->s_draft_len, draft_len, nB * 4, H2D, s));
    OD_CUDA(cudaMemcpyAsync(c->s_q_sel, q_sel, nB * K * 4, H2D, s));
    OD_CUDA(cudaMemcpyAsync(c->s_temperature, temperature, nB * 4, H2D, s));
    OD_CUDA(cudaMemcpyAsync(c->s_seed, seed, nB * 8, H2D, s));
    // Only the rows the step can read cross the bus: logit rows 0..K_b and drafter rows
    // 0..K_b-1 of sequence b (m_b <= K_b). Neighbouring sequences with full proposals
    // merge into one copy; the rest of the staging buffers keeps earlier contents, which
    // no kernel looks at.
    {
        const size_t lrow = (size_t)c->v_p * esz, qrow = (size_t)c->v_q * 4;
        size_t l_from = 0, l_bytes = 0, q_from = 0, q_bytes = 0;   // pending runs (byte offsets)
        for (size_t b = 0; b <= nB; ++b) {
            int32_t kb = 0;
            if (b < nB) { kb = draft_len[b]; kb = kb < 0 ? 0 : (kb > K_max ? K_max : kb); }
            const size_t l_at = b * (K + 1) * lrow, q_at = b * K * qrow;
            if (b == nB || l_from + l_bytes != l_at) {
                if (l_bytes)
                    OD_CUDA(cudaMemcpyAsync((char *)c->s_logits + l_from, (const char *)logits + l_from, l_bytes, H2D, s));
                l_from = l_at; l_bytes = 0;
            }
            if (b == nB || q_from + q_bytes != q_at) {
                if (q_bytes)
                    OD_CUDA(cudaMemcpyAsync((char *)c->s_q_rows + q_from, (const char *)q_rows + q_from, q_bytes, H2D, s));
                q_from = q_at; q_bytes = 0;
            }
            if (b < nB) { l_bytes += (size_t)(kb + 1) * lrow; q_bytes += (size_t)kb * qrow; }
        }
    }
    OD_CUDA(od_launch_map(c, B, K_max, c->s_draft_ids, c->s_draft_len, c->s_q_sel, c->s_tgt_ids,
                          c->s_q_prime, c->s_span_start, c->s_span_len, c->s_m, c->s_tail, nullptr,
                          false /* the copies above are the launches in front */, false, s));
    c->verify_early = true;     // the translation kernel is the launch in front: see od_step
    OD_CUDA(od_launch_verify(c, B, K_max, c->s_logits, logit_dtype, row_stride, seq_stride,
                             c->s_tgt_ids, c->s_q_prime, c->s_span_len, c->s_m, c->s_temperature,
                             c->s_seed, step, c->s_row_max, c->s_row_sum, c->s_p_sel, c->s_ratio,
                             c->s_n_acc, c->s_n_draft, c->s_vflags, s));
    OD_CUDA(od_launch_sample(c, B, K_max, c->s_logits, logit_dtype, row_stride, seq_stride,
                             c->s_row_max, c->s_row_sum, c->s_q_rows, c->s_draft_ids, c->s_tgt_ids,
                             c->s_q_prime, c->s_span_start, c->s_span_len, c->s_m, c->s_tail,
                             c->s_n_acc, c->s_temperature, c->s_seed, step, c->s_token, c->s_mass,
                             c->s_sflags, s));
    if (n_accepted) OD_CUDA(cudaMemcpyAsync(n_accepted, c->s_n_acc, nB * 4, D2H, s));
    if (n_draft_accepted) OD_CUDA(cudaMemcpyAsync(n_draft_accepted, c->s_n_draft, nB * 4, D2H, s));
    if (out_token) OD_CUDA(cudaMemcpyAsync(out_token, c->s_token, nB * 4, D2H, s));
    if (tgt_ids) OD_CUDA(cudaMemcpyAsync(tgt_ids, c->s_tgt_ids, nB * K * 4, D2H, s));
    if (m) OD_CUDA(cudaMemcpyAsync(m, c->s_m, nB * 4, D2H, s));
    if (verify_flags) OD_CUDA(cudaMemcpyAsync(verify_flags, c->s_vflags, nB * 4, D2H, s));
    if (sample_flags) OD_CUDA(cudaMemcpyAsync(sample_flags, c->s_sflags, nB * 4, D2H, s));
    OD_CUDA(cudaStreamSynchronize(s));
    return OD_OK;
}

int64_t od_last_launch_info(const od_ctx *c, int32_t which)
{
    if (!c || which < 0 || which > 3) return -1;
    return c->info[which];
}

const char *od_status_string(int32_t status)
{
    switch (status) {
        case OD_OK: return "ok";
        case OD_ERR_INVALID_ARG: return "invalid argument";
        case OD_ERR_ALIGNMENT: return "logits base or stride not 16-byte aligned";
        case OD_ERR_MAP_NOT_INJECTIVE: return "vocabulary map is not injective";
        case OD_ERR_BAD_CACHE_ENTRY: return "bad n-gram cache entry";
        case OD_ERR_UNSUPPORTED: return "unsupported dtype or size";
        case OD_ERR_CUDA: return "CUDA runtime error";
        case OD_ERR_NOMEM: return "out of memory";
        case OD_ERR_STATE: return "call out of order";
        case OD_ERR_SCRATCH_LIMIT: return "batch too large for the fixed scratch of od_verify_noalloc";
        default: return "unknown status";
    }
}

int32_t od_version(void) { return 100; }

}  // extern "C"
