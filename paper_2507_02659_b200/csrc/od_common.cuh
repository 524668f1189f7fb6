// Shared declarations of the CUDA library: the context, device helpers
// (Philox4x32-10, logit decoding, (max, sum) pair algebra) and the kernel
// launchers implemented in od_map.cu / od_verify.cu / od_sample.cu.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "omnidraft.h"

#define OD_WARP 32
#define OD_GROUP 32                 // slots of one hash-table probe group
#define OD_SAMPLE_TILE 256          // elements of one residual-sampler tile (8 per lane of a warp)
#define OD_SAMPLE_THREADS 256
#define OD_SAMPLE_SMEM_MAX (200 * 1024)  // dynamic shared memory the sampler may ask for: 8 bytes per tile
#define OD_VERIFY_SEG_MAX 64        // most segments (partials) one logit row is cut into
#define OD_VERIFY_MAX_B 2048        // sequences per od_verify launch (longer batches go in slices)

struct od_ctx {
    int device;
    int32_t v_q, v_p, max_batch, max_k;
    int sm_count;

    // vocabulary map (device)
    int32_t *d_vocab_map;           // [v_q]
    int32_t *d_inv_map;             // [v_p], -1 outside the image
    bool have_map;

    // n-gram cache: open addressing over groups of 32 slots
    uint64_t *d_keys;               // [cap], 0 = empty
    int32_t *d_vals;                // [cap]
    int64_t cap;                    // power of two, multiple of 32, or 0

    // online cache (od_cache_configure): per-slot access data of the current table, a
    // second table that od_cache_trim rebuilds into, and the scratch of insert and trim
    bool dyn;
    int32_t dyn_policy;             // 0 = LRU, 1 = LFU
    int64_t dyn_max;                // entries kept by a trim
    int32_t dyn_max_insert;         // largest batch of od_cache_insert
    uint32_t clock;                 // stamp of accesses and insertions
    uint32_t *d_stamp, *d_freq, *d_born;            // [cap]
    uint64_t *d_keys2; int32_t *d_vals2;            // [cap] spare table
    uint32_t *d_stamp2, *d_freq2, *d_born2;
    uint32_t *d_owner;              // [cap] first-wins claims of a batch (0xFFFFFFFF = none)
    int32_t *d_cand_slot;           // [dyn_max_insert]
    void *d_trim;                   // trim / size state (device)
    void *d_trim_lists;             // trim scratch: the live entries' records and two candidate lists, 64 bytes per slot

    // od_verify scratch
    float4 *d_partials;             // [rows][OD_VERIFY_SEG_MAX] (c, sum, max, -), rows of one launch

    // od_sample_residual scratch
    double *d_tile_sums;            // [max_batch * tiles_per_row] value of each tile
    unsigned int *d_samp_ticket;    // [max_batch]
    int32_t tiles_per_row;

    // options
    int64_t opt_verify_grid;        // blocks of the stream kernel (0 = one per multiprocessor)
    int64_t opt_early_inputs;       // the caller promises complete inputs: od_verify reads logits and temperatures, the
                                    // translation kernel the proposal, before griddepcontrol.wait
    int64_t opt_sample_tiles_per_warp;
    int64_t opt_pdl;                // launch with programmatic stream serialization

    // set by the entry points for the verify launch that follows: space A may be streamed early
    bool verify_early;
    bool table_written;             // a kernel that writes the n-gram table was launched since the last translation kernel

    // the last launch on this context was the translation kernel, which lets the next
    // kernel start before its own outputs exist (see od_sample.cu)
    bool last_was_map;

    // last launch info
    int64_t info[4];

    // od_step_host staging (device)
    bool host_reserved;
    int32_t host_dtype;
    void *s_logits;
    float *s_q_rows, *s_q_sel, *s_temperature;
    int32_t *s_draft_ids, *s_draft_len;
    uint64_t *s_seed;
    int32_t *s_tgt_ids, *s_span_start, *s_span_len, *s_m, *s_n_acc, *s_n_draft, *s_token;
    float *s_q_prime, *s_row_max, *s_row_sum, *s_p_sel, *s_ratio, *s_mass;
    uint8_t *s_tail;
    uint32_t *s_vflags, *s_sflags;
};

// ---- launchers ------------------------------------------------------------
cudaError_t od_launch_map(od_ctx *c, int32_t B, int32_t K_max, const int32_t *draft_ids,
                          const int32_t *draft_len, const float *q_sel, int32_t *tgt_ids,
                          float *q_prime, int32_t *span_start, int32_t *span_len, int32_t *m,
                          uint8_t *tail_kind, uint32_t *counters, bool early, bool release_early, cudaStream_t s);

cudaError_t od_launch_verify(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                             int32_t dtype, int64_t row_stride, int64_t seq_stride,
                             const int32_t *tgt_ids, const float *q_prime,
                             const int32_t *span_len, const int32_t *m,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             float *row_max, float *row_sum, float *p_sel, float *ratio,
                             int32_t *n_accepted, int32_t *n_draft_accepted,
                             uint32_t *flags, cudaStream_t s);


// od_step: the streaming pass of step 2 alone (no decide kernel), and what the sampler then needs
// to take step 2's decisions itself: the split of the pass and where step 2's outputs go.
struct od_fused_verify {
    int32_t W, n_chunks, span_min, span_a, seg_warps;
    float *row_max, *row_sum, *p_sel, *ratio;
    int32_t *n_accepted, *n_draft_accepted;
    uint32_t *flags;
};
int32_t od_verify_slice(int32_t K_max, int32_t v_len, int32_t dtype);   // sequences one stream launch takes
cudaError_t od_launch_verify_stream(od_ctx *c, int32_t B, int32_t K_max, const void *logits, int32_t dtype,
                                    int64_t row_stride, int64_t seq_stride, const int32_t *m,
                                    const float *temperature, od_fused_verify *plan, cudaStream_t s);

cudaError_t od_launch_sample(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                             int32_t dtype, int64_t row_stride, int64_t seq_stride,
                             const float *row_max, const float *row_sum, const float *q_rows,
                             const int32_t *draft_ids, const int32_t *tgt_ids,
                             const float *q_prime, const int32_t *span_start,
                             const int32_t *span_len, const int32_t *m,
                             const uint8_t *tail_kind, const int32_t *n_accepted,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             int32_t *out_token, float *resid_mass, uint32_t *flags,
                             cudaStream_t s, const od_fused_verify *fuse = nullptr);

size_t od_sample_smem_bytes(int32_t ntiles);            // dynamic shared memory of the sampler kernel
cudaError_t od_sample_prepare_device(size_t bytes);     // opt in to it where it exceeds the default

// vocabulary shards (columns [shard_lo, shard_lo + shard_len) of the rows on this GPU)
cudaError_t od_launch_verify_shard_stats(od_ctx *c, int32_t B, int32_t K_max, int32_t shard_lo,
                                         int32_t shard_len, const void *logits, int32_t dtype,
                                         int64_t row_stride, int64_t seq_stride, const int32_t *tgt_ids,
                                         const int32_t *m, const float *temperature, float *stats,
                                         cudaStream_t s);
cudaError_t od_launch_verify_shard_finish(od_ctx *c, int32_t B, int32_t K_max, int32_t n_shards,
                                          const float *stats_all, const int32_t *tgt_ids,
                                          const float *q_prime, const int32_t *span_len, const int32_t *m,
                                          const float *temperature, const uint64_t *seed, uint64_t step,
                                          float *row_max, float *row_sum, float *p_sel, float *ratio,
                                          int32_t *n_accepted, int32_t *n_draft_accepted, uint32_t *flags,
                                          cudaStream_t s);
cudaError_t od_launch_sample_shard_mass(od_ctx *c, int32_t B, int32_t K_max, int32_t shard_lo,
                                        int32_t shard_len, const void *logits, int32_t dtype,
                                        int64_t row_stride, int64_t seq_stride, const float *row_max,
                                        const float *row_sum, const float *q_rows, const int32_t *draft_ids,
                                        const int32_t *tgt_ids, const float *q_prime,
                                        const int32_t *span_start, const int32_t *span_len, const int32_t *m,
                                        const uint8_t *tail_kind, const int32_t *n_accepted,
                                        const float *temperature, double *mass, cudaStream_t s);
cudaError_t od_launch_sample_shard_pick(od_ctx *c, int32_t B, int32_t K_max, int32_t n_shards,
                                        int32_t shard_index, int32_t shard_lo, int32_t shard_len,
                                        const double *mass_all, const void *logits, int32_t dtype,
                                        int64_t row_stride, int64_t seq_stride, const float *row_max,
                                        const float *row_sum, const float *q_rows, const int32_t *draft_ids,
                                        const int32_t *tgt_ids, const float *q_prime,
                                        const int32_t *span_start, const int32_t *span_len, const int32_t *m,
                                        const uint8_t *tail_kind, const int32_t *n_accepted,
                                        const float *temperature, const uint64_t *seed, uint64_t step,
                                        int32_t *out_token, float *resid_mass, uint32_t *flags, cudaStream_t s);

cudaError_t od_launch_distill(od_ctx *c, int32_t B, int32_t K_max, const float *q_rows,
                              const int32_t *draft_ids, const int32_t *tgt_ids, const int32_t *span_start,
                              const int32_t *span_len, const int32_t *m, const void *logits, int32_t dtype,
                              int64_t row_stride, int64_t seq_stride, const float *row_max,
                              const float *row_sum, const float *p_sel, const float *temperature,
                              float lambda, int32_t lambda_mode, float *loss, float *grad, cudaStream_t s);

void od_cache_free_dynamic(od_ctx *c);   // frees what od_cache_configure allocated beyond keys / vals

cudaError_t od_launch_exit(int32_t B, int32_t K_max, const float *head_logits, const int32_t *avail_len,
                           float gamma, int32_t *draft_len, float *reject_prob, uint32_t *flags,
                           cudaStream_t s);

// 64-bit key of a run of draft ids: (id + 1) in 16 bits per position, first id
// in the low bits. Never 0 for a non-empty run.
__host__ __device__ inline uint64_t od_pack_run(const int32_t *ids, int len)
{
    uint64_t k = 0;
    for (int j = 0; j < len; ++j) k |= (uint64_t)(uint32_t)(ids[j] + 1) << (16 * j);
    return k;
}

// 64-bit finaliser of MurmurHash3 (Appleby, public domain): spreads the packed
// key over the table's groups.
__host__ __device__ inline uint64_t od_hash64(uint64_t h)
{
    h ^= h >> 33; h *= 0xff51afd7ed558ccdULL;
    h ^= h >> 33; h *= 0xc4ceb9fe1a85ec53ULL;
    h ^= h >> 33;
    return h;
}

#ifdef __CUDACC__
// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) ----------------------
__device__ __forceinline__ uint32_t od_philox_word0(uint32_t c0, uint32_t c1, uint32_t c2,
                                                    uint32_t c3, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}

// uniform in [0,1) on the 24-bit grid for (seed, step, position, tag)
__device__ __forceinline__ float od_uniform(uint64_t seed, uint64_t step, uint32_t position,
                                            uint32_t tag)
{
    uint32_t w = od_philox_word0((uint32_t)step, (uint32_t)(step >> 32), position, tag,
                                 (uint32_t)seed, (uint32_t)(seed >> 32));
    return (float)(w >> 8) * (1.0f / 16777216.0f);
}

__device__ __forceinline__ float od_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packed fp32 pairs (one instruction for two lanes of arithmetic on sm_100).
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// acc += (exp2(lo*scale - c), exp2(hi*scale - c))
__device__ __forceinline__ uint64_t f2_exp_acc(uint64_t acc, float lo, float hi, uint64_t scale2, uint64_t nc2)
{
    float e0, e1;
    f2_unpack(f2_fma(f2_pack(lo, hi), scale2, nc2), e0, e1);
    return f2_add(acc, f2_pack(od_ex2(e0), od_ex2(e1)));
}

// (max, sum) of exp2((x - max) * scale): merge two partial pairs
__device__ __forceinline__ void od_pair_merge(float &m, float &s, float m2, float s2, float scale)
{
    float nm = fmaxf(m, m2);
    s = s * od_ex2((m - nm) * scale) + s2 * od_ex2((m2 - nm) * scale);
    m = nm;
}

__device__ __forceinline__ float od_bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float od_bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

template <int DTYPE>
__device__ __forceinline__ float od_load_logit(const void *row, int64_t t)
{
    if (DTYPE == OD_F32) return __ldg((const float *)row + t);
    uint16_t h = __ldg((const unsigned short *)row + t);
    return __uint_as_float((uint32_t)h << 16);
}
#endif  // __CUDACC__
