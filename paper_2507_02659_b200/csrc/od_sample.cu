// Step 3: the extra token of a verification step: a draw from the normalised
// residual max(0, p - q') at the first rejection, with q'(.) of Eq. (2), or
// from p itself (the free token) when every proposal was accepted (notation
// paragraph of Section 3; Section 3.1, Eq. (2); Algorithm 1, rejection and
// free-token lines).
//
// Inverse-CDF sampling in target-id order over tiles of 256 ids (8 consecutive
// ids per lane of one warp, so a tile needs shuffles only, no block barrier):
//   pass 1  every warp computes r(t) for its run of tiles of row j = n_b and
//           stores one fp64 sum per tile;
//   ticket  blocks never wait for each other: the block that draws the
//           sequence's last ticket continues alone;
//   pass 2  that block scans the tile sums in parallel (R = total, target =
//           u * R), finds the tile in which the running sum crosses the target,
//           and one warp recomputes that tile (L2-resident) and scans inside it.
// r(t) is evaluated in fp32 exactly the same way in both passes; all sums and
// scans are fp64 in a fixed order, so the result is reproducible and the only
// difference to exact arithmetic is the fp32 rounding of the individual r(t).
#include <float.h>

#include "od_common.cuh"

namespace {

constexpr int WARPS = OD_SAMPLE_THREADS / 32;
constexpr int EPT = OD_SAMPLE_TILE / 32;                  // ids per lane per tile (8)

struct SampleArgs {
    const void *logits;
    int64_t row_stride, seq_stride;
    int32_t B, K_max, v_p, v_q;
    int32_t ntiles, tiles_per_warp;
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

// what one sequence's warps need to evaluate r(t)
struct SeqState {
    const char *row;
    const float *q_row;
    float M, S, scale;
    bool residual;
    int32_t ngram_token, prefix_token;
    float ngram_prob, prefix_val;
};

// Values are carried UNNORMALISED: with e(t) = exp2((x_t - M)*scale) = p(t)*S,
//   residual   r'(t) = max(0, e(t) - q'(t)*S) = S * max(0, p(t) - q'(t))
//   free token r'(t) = e(t)
// so one multiplication by 1/S at the very end replaces one per element, and the
// inverse-CDF pick (target = u * sum r') is unchanged by the common factor.
__device__ __forceinline__ float resid_of(const SeqState &q, float x, float qq)
{
    return fmaxf(0.f, fmaf(-qq, q.S, od_ex2((x - q.M) * q.scale)));
}

// r'(t) of the EPT consecutive ids this lane owns in `tile`; ids >= v_p give 0
template <int DTYPE>
__device__ __forceinline__ void tile_values(const SeqState &q, const SampleArgs &a, bool residual,
                                            int tile, int lane, float *r)
{
    const int t0 = tile * OD_SAMPLE_TILE + lane * EPT;
    if (t0 + EPT <= a.v_p) {
        float x[EPT];
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
            const int32_t d[EPT] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
            float qq[EPT];
#pragma unroll
            for (int e = 0; e < EPT; ++e) qq[e] = d[e] >= 0 ? __ldg(q.q_row + d[e]) : 0.f;
#pragma unroll
            for (int e = 0; e < EPT; ++e) r[e] = resid_of(q, x[e], qq[e]);
        } else {
#pragma unroll
            for (int e = 0; e < EPT; ++e) r[e] = od_ex2((x[e] - q.M) * q.scale);
        }
    } else {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int t = t0 + e;
            r[e] = 0.f;
            if (t < a.v_p) {
                const float xv = od_load_logit<DTYPE>(q.row, t);
                if (residual) {
                    const int32_t dv = __ldg(a.inv_map + t);
                    r[e] = resid_of(q, xv, dv >= 0 ? __ldg(q.q_row + dv) : 0.f);
                } else {
                    r[e] = od_ex2((xv - q.M) * q.scale);
                }
            }
        }
    }
    if (residual) {
        // Eq. (2): the two ids whose q' is not the drafter's row. Only the lane that
        // owns such an id redoes it (prefix sub-token first, the n-gram token last).
        const int dp = q.prefix_token - t0, dn = q.ngram_token - t0;
        if ((unsigned)dp < (unsigned)EPT && q.prefix_token < a.v_p) {
            const float v = resid_of(q, od_load_logit<DTYPE>(q.row, q.prefix_token), q.prefix_val);
#pragma unroll
            for (int e = 0; e < EPT; ++e) r[e] = e == dp ? v : r[e];
        }
        if ((unsigned)dn < (unsigned)EPT && q.ngram_token < a.v_p) {
            const float v = resid_of(q, od_load_logit<DTYPE>(q.row, q.ngram_token), q.ngram_prob);
#pragma unroll
            for (int e = 0; e < EPT; ++e) r[e] = e == dn ? v : r[e];
        }
    }
}

// a lane's eight values are added in fp32 in index order (both passes do exactly
// this); everything across lanes and tiles is fp64
__device__ __forceinline__ double lane_sum(const float *r)
{
    float s = r[0];
#pragma unroll
    for (int e = 1; e < EPT; ++e) s += r[e];
    return (double)s;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    return v;
}

// tile sums of tiles [t_lo, t_hi) by one warp: index order inside a lane, xor
// tree across the lanes
template <int DTYPE>
__device__ __forceinline__ void warp_tiles(const SeqState &q, const SampleArgs &a, bool residual,
                                           int t_lo, int t_hi, int lane, double *sums)
{
    int tile = t_lo;
    for (; tile + 2 <= t_hi; tile += 2) {                  // two tiles in flight
        float r0[EPT], r1[EPT];
        tile_values<DTYPE>(q, a, residual, tile, lane, r0);
        tile_values<DTYPE>(q, a, residual, tile + 1, lane, r1);
        const double s0 = warp_sum(lane_sum(r0)), s1 = warp_sum(lane_sum(r1));
        if (lane == 0) { sums[tile] = s0; sums[tile + 1] = s1; }
    }
    if (tile < t_hi) {
        float r0[EPT];
        tile_values<DTYPE>(q, a, residual, tile, lane, r0);
        const double s0 = warp_sum(lane_sum(r0));
        if (lane == 0) sums[tile] = s0;
    }
    __threadfence();                                       // the sums are read by another block
}

template <int DTYPE>
__global__ void __launch_bounds__(OD_SAMPLE_THREADS, 4)
od_sample_kernel(const SampleArgs a)
{
    __shared__ double s_warp[WARPS];
    __shared__ unsigned int s_last;
    __shared__ int s_tile, s_lastmass;
    __shared__ double s_before, s_total;

    // n_accepted and the row statistics come from the verification kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");

    const int b = blockIdx.y;
    const int K = a.K_max;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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
    q.S = a.row_sum[b * (K + 1) + j];
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
    const int ntiles = a.ntiles;
    double *sums = a.tile_sums + (size_t)b * ntiles;
    {
        const int t_lo = (blockIdx.x * WARPS + warp) * a.tiles_per_warp;
        int t_hi = t_lo + a.tiles_per_warp;
        if (t_hi > ntiles) t_hi = ntiles;
        if (t_lo < t_hi) warp_tiles<DTYPE>(q, a, q.residual, t_lo, t_hi, lane, sums);
    }
    __syncthreads();
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
    const int per = (ntiles + OD_SAMPLE_THREADS - 1) / OD_SAMPLE_THREADS;
    const int my_lo = threadIdx.x * per;
    const int my_hi = my_lo + per < ntiles ? my_lo + per : ntiles;
    const volatile double *vs = sums;
    double target = 0.0;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // exclusive scan of the tile sums: thread i owns `per` consecutive tiles
        double loc = 0.0;
        for (int t = my_lo; t < my_hi; ++t) loc += vs[t];
        double inc = loc;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double v = __shfl_up_sync(0xFFFFFFFFu, inc, off);
            if (lane >= off) inc += v;
        }
        if (lane == 31) s_warp[warp] = inc;
        if (threadIdx.x == 0) { s_tile = 0x7FFFFFFF; s_lastmass = -1; }
        __syncthreads();
        double base = 0.0;
        for (int w = 0; w < warp; ++w) base += s_warp[w];
        if (threadIdx.x == OD_SAMPLE_THREADS - 1) s_total = base + inc;
        __syncthreads();
        const double R = s_total;
        if (R > 0.0) {
            target = (double)u * R;
            double c = base + inc - loc;
            int last = -1;
            for (int t = my_lo; t < my_hi; ++t) {
                const double v = vs[t];
                if (v > 0.0) last = t;
                if (c + v > target) { atomicMin(&s_tile, t); break; }   // first crossing of this run
                c += v;
            }
            if (last >= 0) atomicMax(&s_lastmass, last);
        }
        __syncthreads();
        if (R > 0.0) {
            // cumulative sums never decrease, so the smallest reported tile is the crossing;
            // if rounding hid it, take the last tile that has mass
            const int t_pick = s_tile != 0x7FFFFFFF ? s_tile : s_lastmass;
            __syncthreads();
            if (t_pick >= my_lo && t_pick < my_hi) {        // its owner publishes the sum before it
                double c = base + inc - loc;
                for (int t = my_lo; t < t_pick; ++t) c += vs[t];
                s_before = c;
                s_tile = t_pick;
            }
            __syncthreads();
            break;
        }
        if (attempt == 1) {
            if (threadIdx.x == 0) s_tile = -1;
            __syncthreads();
            break;
        }
        // no residual mass: draw from p_j instead (rare; this block redoes the row)
        residual = false;
        flags |= OD_SF_ZERO_MASS;
        for (int t_lo = warp * 2; t_lo < ntiles; t_lo += WARPS * 2)
            warp_tiles<DTYPE>(q, a, false, t_lo, t_lo + 2 < ntiles ? t_lo + 2 : ntiles, lane, sums);
        __syncthreads();
    }
    if (s_tile < 0 || s_tile == 0x7FFFFFFF) {       // no mass at all (non-finite input)
        if (threadIdx.x == 0) {
            a.out_token[b] = -1; a.resid_mass[b] = (float)(s_total / (double)q.S);
            a.flags[b] = flags | OD_SF_ZERO_MASS;
            a.ticket[b] = 0;
        }
        return;
    }
    if (warp != 0) return;

    // ---- warp 0 scans inside the chosen tile ----
    const int tile = s_tile;
    const double Rn = s_total;                      // unnormalised total
    float r[EPT];
    tile_values<DTYPE>(q, a, residual, tile, lane, r);
    const double mine = lane_sum(r);
    double incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += v;
    }
    const double base = s_before + (incl - mine);   // sum before this lane's first id
    const int t0 = tile * OD_SAMPLE_TILE + lane * EPT;
    int my_pick = 0x7FFFFFFF, my_last = -1;
    double lo = 0.0, hi = 0.0;
    float run = 0.f;                                // same fp32 order as lane_sum
    double c = base;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        run = e == 0 ? r[0] : run + r[e];
        const double nc = base + (double)run;
        if (r[e] > 0.f) my_last = t0 + e;
        if (my_pick == 0x7FFFFFFF && nc > target) { my_pick = t0 + e; lo = c; hi = nc; }
        c = nc;
    }
    int pick = my_pick, last = my_last;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        pick = min(pick, __shfl_xor_sync(0xFFFFFFFFu, pick, off));
        last = max(last, __shfl_xor_sync(0xFFFFFFFFu, last, off));
    }
    const float R = (float)(Rn / (double)q.S);      // residual mass (1 for the free token)
    if (pick != 0x7FFFFFFF) {
        if (my_pick == pick) {                      // exactly one lane owns the picked id
            const double margin = fmin(target - lo, hi - target);
            if (margin <= OD_TAU_SAMPLE * Rn) flags |= OD_SF_BOUNDARY;
            a.out_token[b] = pick;
            a.resid_mass[b] = R;
            a.flags[b] = flags;
            a.ticket[b] = 0;
        }
    } else if (lane == 0) {
        // rounding: target beyond the tile's last edge
        a.out_token[b] = last;
        a.resid_mass[b] = R;
        a.flags[b] = flags | OD_SF_BOUNDARY | (last < 0 ? OD_SF_ZERO_MASS : 0u);
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
    int64_t tpw = c->opt_sample_tiles_per_warp;
    if (tpw <= 0) {
        // one resident wave (four 256-thread blocks per SM) over the whole batch
        const int64_t want = (int64_t)c->sm_count * 4;
        int64_t per_row = want / B;
        if (per_row < 1) per_row = 1;
        tpw = (ntiles + per_row * WARPS - 1) / (per_row * WARPS);
        if (tpw < 1) tpw = 1;
    }
    const int64_t tiles_per_block = tpw * WARPS;
    const int blocks_x = (int)((ntiles + tiles_per_block - 1) / tiles_per_block);
    SampleArgs a;
    a.logits = logits; a.row_stride = row_stride; a.seq_stride = seq_stride;
    a.B = B; a.K_max = K_max; a.v_p = c->v_p; a.v_q = c->v_q;
    a.ntiles = ntiles; a.tiles_per_warp = (int32_t)tpw;
    a.row_max = row_max; a.row_sum = row_sum; a.q_rows = q_rows;
    a.draft_ids = draft_ids; a.tgt_ids = tgt_ids; a.q_prime = q_prime;
    a.span_start = span_start; a.span_len = span_len; a.m = m; a.tail_kind = tail_kind;
    a.n_accepted = n_accepted; a.temperature = temperature; a.seed = seed; a.step = step;
    a.vocab_map = c->d_vocab_map; a.inv_map = c->d_inv_map;
    a.out_token = out_token; a.resid_mass = resid_mass; a.flags = flags;
    a.tile_sums = c->d_tile_sums; a.ticket = c->d_samp_ticket;
    c->info[2] = (int64_t)blocks_x * B;
    c->info[3] = tpw;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks_x, (unsigned)B);
    cfg.blockDim = dim3(OD_SAMPLE_THREADS);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->opt_pdl ? 1 : 0;
    return dtype == OD_BF16 ? cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_BF16>, a)
                            : cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_F32>, a);
}
