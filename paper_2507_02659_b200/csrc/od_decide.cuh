// What od_verify's two kernels and the sampler of od_step share: where the streaming pass
// leaves the partial statistics of a row, how they are merged, and the acceptance decision of
// one position (Section 3.1, acceptance ratio; Algorithm 1, rejection-sampling line).
#pragma once

#include <float.h>

#include "od_common.cuh"

// The split of the streaming pass (see od_verify.cu): enough to find a row's partials.
struct StreamPlan {
    int32_t W;                      // 512-byte units per row
    int32_t n_chunks;               // blocks of the stream grid
    int32_t span_min;               // smallest span of space B
    int32_t span_a;                 // units of space A per block
    int32_t seg_warps;              // warps of a stream-kernel block: partials per block segment
    const float4 *partials;         // [row slot][OD_VERIFY_SEG_MAX] (c, sum, max, -)
};

// How many blocks hold pieces of flat row `rho` of a space whose blocks take
// `span` units each.
__device__ __forceinline__ int row_segments(uint32_t rho, uint32_t W, uint32_t span)
{
    return (int)(((rho + 1) * W - 1) / span - rho * W / span + 1);
}

__device__ __forceinline__ uint32_t span_of_space_b(uint32_t rows_b, uint32_t W, uint32_t n_chunks, uint32_t span_min)
{
    const uint32_t span = (rows_b * W + n_chunks - 1) / n_chunks;
    return span < span_min ? span_min : span;
}

__device__ __forceinline__ int clamp_m(int mb, int K_max) { return mb < 0 ? 0 : (mb > K_max ? K_max : mb); }

// (c, s) pairs: s counts exp2(x*scale - c)
__device__ __forceinline__ void pair_merge(float &c, float &s, float c2, float s2)
{
    const float cm = fmaxf(c, c2);
    s = s * od_ex2(c - cm) + s2 * od_ex2(c2 - cm);
    c = cm;
}

// all lanes end with the merged (c, s, mx): one rescale per lane, then plain reductions
__device__ __forceinline__ void warp_merge(float &c, float &s, float &mx)
{
    float cm = c;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        cm = fmaxf(cm, __shfl_xor_sync(0xFFFFFFFFu, cm, off));
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
    }
    s *= od_ex2(c - cm);
    c = cm;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
}

// Partials of row r of sequence b (`before` = rows 1.. of the sequences in front of b,
// `total` = of the whole batch): how many block segments the row was cut into.
__device__ __forceinline__ int row_partial_segments(const StreamPlan &p, int b, int r, int before, int total)
{
    if (r == 0) return row_segments((uint32_t)b, (uint32_t)p.W, (uint32_t)p.span_a);
    return row_segments((uint32_t)(before + r - 1), (uint32_t)p.W,
                        span_of_space_b((uint32_t)total, (uint32_t)p.W, (uint32_t)p.n_chunks, (uint32_t)p.span_min));
}

// One warp merges the partials of a row (nseg block segments): every lane ends with the
// row's (c, s, mx). The order is fixed, so every caller gets the same bits.
__device__ __forceinline__ void merge_row_partials(const StreamPlan &p, int row_slot, int nseg, int lane,
                                                   float &c, float &s, float &mx)
{
    const float4 *pp = p.partials + (size_t)row_slot * OD_VERIFY_SEG_MAX;
    // at most OD_VERIFY_SEG_MAX = 64 partials: two per lane, both requested before either is used
    const int n = nseg * p.seg_warps;
    float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f), v1 = v0;
    if (lane < n) v0 = __ldcg(pp + lane);
    if (lane + 32 < n) v1 = __ldcg(pp + lane + 32);
    c = -FLT_MAX; s = 0.f; mx = -INFINITY;
    if (lane < n) { pair_merge(c, s, v0.x, v0.y); mx = fmaxf(mx, v0.z); }
    if (lane + 32 < n) { pair_merge(c, s, v1.x, v1.y); mx = fmaxf(mx, v1.z); }
    warp_merge(c, s, mx);
}

// Row sum relative to the exact maximum M = mx from the merged (c, s): removes the rounding of c.
__device__ __forceinline__ float row_sum_of(float c, float s, float mx, float scale)
{
    return s * od_ex2(fmaf(-mx, scale, c));
}

// The acceptance test of one position: p(t_i), min(1, p/q'), accept iff u < ratio.
struct Acceptance {
    float p, ratio;
    bool accept, boundary;
};
__device__ __forceinline__ Acceptance accept_position(float M, float S, float scale, bool t_ok, float x_t, float q,
                                                      float u)
{
    Acceptance r;
    r.p = t_ok ? od_ex2((x_t - M) * scale) / S : 0.f;
    r.ratio = (q <= r.p) ? 1.f : r.p / q;
    r.accept = u < r.ratio;
    r.boundary = fabsf(u - r.ratio) <= OD_TAU_ACCEPT;
    return r;
}
