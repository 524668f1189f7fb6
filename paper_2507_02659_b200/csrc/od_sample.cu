// Step 3: the extra token of a verification step: a draw from the normalised
// residual max(0, p - q') at the first rejection, with q'(.) of Eq. (2), or
// from p itself (the free token) when every proposal was accepted (notation
// paragraph of Section 3; Section 3.1, Eq. (2); Algorithm 1, rejection and
// free-token lines).
//
// Inverse-CDF sampling in target-id order, organised as tiles of 2048 ids:
//   pass 1  every block computes r(t) for its tiles of row j = n_b and stores
//           one fp64 sum per tile;
//   ticket  blocks never wait for each other: the block that draws the
//           sequence's last ticket continues alone;
//   pass 2  that block scans the tile sums (R = total, target = u * R), finds
//           the tile in which the running sum crosses the target, recomputes
//           that one tile (2048 ids, L2-resident) and scans inside it.
// r(t) is evaluated in fp32 exactly the same way in both passes; all sums and
// scans are fp64 in a fixed order, so the result is reproducible and the only
// difference to exact arithmetic is the fp32 rounding of the individual r(t).
#include <float.h>

#include "od_common.cuh"

namespace {

struct SampleArgs {
    const void *logits;
    int64_t row_stride, seq_stride;
    int32_t B, K_max, v_p, v_q;
    int32_t tiles_per_row, tiles_per_block;
    const float *row_max, *row_sum, *q_rows;
    const int32_t *draft_ids, *tgt_ids;
    const float *q_prime;
    const int32_t *span_start, *span_len, *m;
    const uint8_t *tail_kind;
    const int32_t *n_accepted;
    const float *temperature;
    const uint64_t *seed;
    uint64_t step;
    const int32_t *vocab_map, *inv_map;
    int32_t *out_token;
    float *resid_mass;
    uint32_t *flags;
    double *tile_sums;
    unsigned int *ticket;
};

// what one sequence's blocks need to evaluate r(t)
struct SeqState {
    const char *row;
    const float *q_row;
    float M, invS, scale;
    bool residual;
    int32_t ngram_token, prefix_token;
    float ngram_prob, prefix_val;
};

constexpr int EPT = OD_SAMPLE_TILE / OD_SAMPLE_THREADS;   // elements per thread per tile (8)

template <int DTYPE>
__device__ __forceinline__ float r_of(const SeqState &q, const int32_t *__restrict__ inv_map,
                                      bool residual, int64_t t, float x, int32_t d)
{
    float p = od_ex2((x - q.M) * q.scale) * q.invS;
    if (!residual) return p;
    float qq = d >= 0 ? __ldg(q.q_row + d) : 0.f;
    if (t == q.prefix_token) qq = q.prefix_val;
    if (t == q.ngram_token) qq = q.ngram_prob;
    return fmaxf(0.f, p - qq);
}

// r(t) of the EPT consecutive ids a thread owns in `tile`; ids >= v_p give 0
template <int DTYPE>
__device__ __forceinline__ void tile_values(const SeqState &q, const SampleArgs &a, bool residual,
                                            int tile, float *r)
{
    const int64_t t0 = (int64_t)tile * OD_SAMPLE_TILE + (int64_t)threadIdx.x * EPT;
    float x[EPT];
    int32_t d[EPT];
    if (t0 + EPT <= a.v_p) {
        if (DTYPE == OD_BF16) {
            const uint4 v = __ldg((const uint4 *)(q.row + (size_t)t0 * 2));
            x[0] = od_bf16_lo(v.x); x[1] = od_bf16_hi(v.x); x[2] = od_bf16_lo(v.y); x[3] = od_bf16_hi(v.y);
            x[4] = od_bf16_lo(v.z); x[5] = od_bf16_hi(v.z); x[6] = od_bf16_lo(v.w); x[7] = od_bf16_hi(v.w);
        } else {
            const float4 v0 = __ldg((const float4 *)(q.row + (size_t)t0 * 4));
            const float4 v1 = __ldg((const float4 *)(q.row + (size_t)t0 * 4) + 1);
            x[0] = v0.x; x[1] = v0.y; x[2] = v0.z; x[3] = v0.w;
            x[4] = v1.x; x[5] = v1.y; x[6] = v1.z; x[7] = v1.w;
        }
        if (residual) {
            const int4 i0 = __ldg((const int4 *)(a.inv_map + t0));
            const int4 i1 = __ldg((const int4 *)(a.inv_map + t0) + 1);
            d[0] = i0.x; d[1] = i0.y; d[2] = i0.z; d[3] = i0.w;
            d[4] = i1.x; d[5] = i1.y; d[6] = i1.z; d[7] = i1.w;
        }
#pragma unroll
        for (int e = 0; e < EPT; ++e) r[e] = r_of<DTYPE>(q, a.inv_map, residual, t0 + e, x[e], residual ? d[e] : -1);
    } else {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int64_t t = t0 + e;
            if (t < a.v_p) {
                const float xv = od_load_logit<DTYPE>(q.row, t);
                const int32_t dv = residual ? __ldg(a.inv_map + t) : -1;
                r[e] = r_of<DTYPE>(q, a.inv_map, residual, t, xv, dv);
            } else {
                r[e] = 0.f;
            }
        }
    }
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, off);
    return v;
}

// sum of one tile, valid in thread 0; fixed order (index order inside a thread,
// shuffle tree inside a warp, warps in order)
template <int DTYPE>
__device__ double tile_sum(const SeqState &q, const SampleArgs &a, bool residual, int tile,
                           double *s_warp)
{
    float r[EPT];
    tile_values<DTYPE>(q, a, residual, tile, r);
    double s = 0.0;
#pragma unroll
    for (int e = 0; e < EPT; ++e) s += (double)r[e];
    s = warp_sum(s);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) s_warp[warp] = s;
    __syncthreads();
    double tot = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < OD_SAMPLE_THREADS / 32; ++w) tot += s_warp[w];
    return tot;
}

template <int DTYPE>
__global__ void __launch_bounds__(OD_SAMPLE_THREADS)
od_sample_kernel(const SampleArgs a)
{
    __shared__ double s_warp[OD_SAMPLE_THREADS / 32];
    __shared__ unsigned int s_last;
    __shared__ int s_tile, s_pick, s_lastpos;
    __shared__ double s_before, s_total, s_target, s_lo, s_hi;

    const int b = blockIdx.y;
    const int K = a.K_max;
    int mb = a.m[b];
    mb = mb < 0 ? 0 : (mb > K ? K : mb);
    int j = a.n_accepted[b];
    j = j < 0 ? 0 : (j > mb ? mb : j);
    const bool stop = a.tail_kind[b] == OD_TAIL_UNMAPPED_STOP;
    const float T = a.temperature[b];
    if (!(T > 0.f)) {                              // every block of the sequence leaves here
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            a.out_token[b] = -1; a.resid_mass[b] = 0.f; a.flags[b] = OD_SF_BAD_TEMPERATURE;
        }
        return;
    }
    const size_t esz = DTYPE == OD_BF16 ? 2 : 4;
    SeqState q;
    q.row = (const char *)a.logits + ((size_t)b * a.seq_stride + (size_t)j * a.row_stride) * esz;
    q.M = a.row_max[b * (K + 1) + j];
    q.invS = 1.f / a.row_sum[b * (K + 1) + j];
    q.scale = 1.4426950408889634f / T;
    q.residual = (j < mb) || stop;
    q.ngram_token = -1; q.prefix_token = -1; q.ngram_prob = 0.f; q.prefix_val = 0.f;
    q.q_row = a.q_rows;
    if (q.residual) {
        const size_t o = (size_t)b * K + j;
        int s0 = a.span_start[o];
        s0 = s0 < 0 ? 0 : (s0 >= K ? K - 1 : s0);
        q.q_row = a.q_rows + ((size_t)b * K + s0) * a.v_q;
        const int len = j < mb ? a.span_len[o] : 1;
        if (len >= 2) {
            q.ngram_token = a.tgt_ids[o];
            q.ngram_prob = a.q_prime[o];
            const int32_t d1 = a.draft_ids[(size_t)b * K + s0];
            if (d1 >= 0 && d1 < a.v_q) {
                q.prefix_token = __ldg(a.vocab_map + d1);
                q.prefix_val = __ldg(q.q_row + d1) - q.ngram_prob;
            }
        }
    }

    // ---- pass 1: one fp64 sum per tile ----
    const int ntiles = a.tiles_per_row;
    double *sums = a.tile_sums + (size_t)b * ntiles;
    const int t_lo = blockIdx.x * a.tiles_per_block;
    int t_hi = t_lo + a.tiles_per_block;
    if (t_hi > ntiles) t_hi = ntiles;
    for (int tile = t_lo; tile < t_hi; ++tile) {
        const double s = tile_sum<DTYPE>(q, a, q.residual, tile, s_warp);
        if (threadIdx.x == 0) sums[tile] = s;
    }
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(a.ticket + b, 1u) == gridDim.x - 1 ? 1u : 0u;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // ---- pass 2 (one block per sequence) ----
    bool residual = q.residual;
    uint32_t flags = residual ? 0u : OD_SF_BONUS;
    const float u = od_uniform(a.seed[b], a.step, (uint32_t)j, 1u);
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (threadIdx.x == 0) {
            const volatile double *vs = sums;
            double tot = 0.0;
            for (int t = 0; t < ntiles; ++t) tot += vs[t];
            s_total = tot;
            s_tile = -1;
            if (tot > 0.0) {
                const double target = (double)u * tot;
                double c = 0.0, before = 0.0;
                int pick = -1;
                for (int t = 0; t < ntiles; ++t) {          // same order as the total above
                    const double nc = c + vs[t];
                    if (nc > target) { pick = t; before = c; break; }
                    c = nc;
                }
                if (pick < 0) {                             // unreachable for u < 1; stay safe
                    c = 0.0;
                    for (int t = 0; t < ntiles; ++t) {
                        if (vs[t] > 0.0) { pick = t; before = c; }
                        c += vs[t];
                    }
                }
                s_tile = pick; s_before = before; s_target = target;
            }
            s_pick = 0x7FFFFFFF; s_lastpos = -1;
        }
        __syncthreads();
        if (s_tile >= 0) break;
        if (attempt == 1) break;
        // no residual mass: draw from p_j instead (rare; this block redoes the row)
        residual = false;
        flags |= OD_SF_ZERO_MASS;
        for (int tile = 0; tile < ntiles; ++tile) {
            const double s = tile_sum<DTYPE>(q, a, false, tile, s_warp);
            if (threadIdx.x == 0) sums[tile] = s;
        }
        __syncthreads();
    }
    if (s_tile < 0) {                               // no mass at all (non-finite input)
        if (threadIdx.x == 0) {
            a.out_token[b] = -1; a.resid_mass[b] = (float)s_total; a.flags[b] = flags | OD_SF_ZERO_MASS;
            a.ticket[b] = 0;
        }
        return;
    }

    // scan inside the chosen tile
    const int tile = s_tile;
    float r[EPT];
    tile_values<DTYPE>(q, a, residual, tile, r);
    double mine = 0.0;
#pragma unroll
    for (int e = 0; e < EPT; ++e) mine += (double)r[e];
    // exclusive scan of the per-thread sums in thread order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    double base = s_before;
    for (int w = 0; w < warp; ++w) base += s_warp[w];
    double c = base + (incl - mine);
    const double target = s_target;
    const int64_t t0 = (int64_t)tile * OD_SAMPLE_TILE + (int64_t)threadIdx.x * EPT;
    int my_pick = -1, my_last = -1;
    double lo = 0.0, hi = 0.0;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        const double nc = c + (double)r[e];
        if (r[e] > 0.f) my_last = (int)(t0 + e);
        if (my_pick < 0 && nc > target) { my_pick = (int)(t0 + e); lo = c; hi = nc; }
        c = nc;
    }
    if (my_pick >= 0) atomicMin(&s_pick, my_pick);
    if (my_last >= 0) atomicMax(&s_lastpos, my_last);
    __syncthreads();
    if (my_pick >= 0 && my_pick == s_pick) { s_lo = lo; s_hi = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        int tok;
        const double R = s_total;
        if (s_pick != 0x7FFFFFFF) {
            tok = s_pick;
            const double margin = fmin(target - s_lo, s_hi - target);
            if (margin <= OD_TAU_SAMPLE * R) flags |= OD_SF_BOUNDARY;
        } else {
            tok = s_lastpos;                        // rounding: target beyond the tile's last edge
            flags |= OD_SF_BOUNDARY;
        }
        a.out_token[b] = tok;
        a.resid_mass[b] = (float)R;
        a.flags[b] = flags;
        a.ticket[b] = 0;
    }
}

}  // namespace

cudaError_t od_launch_sample(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                             int32_t dtype, int64_t row_stride, int64_t seq_stride,
                             const float *row_max, const float *row_sum, const float *q_rows,
                             const int32_t *draft_ids, const int32_t *tgt_ids,
                             const float *q_prime, const int32_t *span_start,
                             const int32_t *span_len, const int32_t *m,
                             const uint8_t *tail_kind, const int32_t *n_accepted,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             int32_t *out_token, float *resid_mass, uint32_t *flags,
                             cudaStream_t s)
{
    if (B == 0) return cudaSuccess;
    const int ntiles = c->tiles_per_row;
    int64_t tpb = c->opt_sample_tiles_per_block;
    if (tpb <= 0) {
        // aim at ~8 blocks per SM over the whole batch
        const int64_t want = (int64_t)c->sm_count * 8;
        const int64_t per_row = (want + B - 1) / B;
        tpb = (ntiles + per_row - 1) / per_row;
        if (tpb < 1) tpb = 1;
    }
    if (tpb > ntiles) tpb = ntiles;
    const int blocks_x = (int)((ntiles + tpb - 1) / tpb);
    SampleArgs a;
    a.logits = logits; a.row_stride = row_stride; a.seq_stride = seq_stride;
    a.B = B; a.K_max = K_max; a.v_p = c->v_p; a.v_q = c->v_q;
    a.tiles_per_row = ntiles; a.tiles_per_block = (int32_t)tpb;
    a.row_max = row_max; a.row_sum = row_sum; a.q_rows = q_rows;
    a.draft_ids = draft_ids; a.tgt_ids = tgt_ids; a.q_prime = q_prime;
    a.span_start = span_start; a.span_len = span_len; a.m = m; a.tail_kind = tail_kind;
    a.n_accepted = n_accepted; a.temperature = temperature; a.seed = seed; a.step = step;
    a.vocab_map = c->d_vocab_map; a.inv_map = c->d_inv_map;
    a.out_token = out_token; a.resid_mass = resid_mass; a.flags = flags;
    a.tile_sums = c->d_tile_sums; a.ticket = c->d_samp_ticket;
    dim3 grid((unsigned)blocks_x, (unsigned)B);
    c->info[2] = (int64_t)blocks_x * B;
    c->info[3] = tpb;
    if (dtype == OD_BF16)
        od_sample_kernel<OD_BF16><<<grid, OD_SAMPLE_THREADS, 0, s>>>(a);
    else
        od_sample_kernel<OD_F32><<<grid, OD_SAMPLE_THREADS, 0, s>>>(a);
    return cudaGetLastError();
}
