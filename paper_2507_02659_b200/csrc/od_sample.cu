// Step 3: the extra token of a verification step: a draw from the normalised
// residual max(0, p - q') at the first rejection, with q'(.) of Eq. (2), or
// from p itself (the free token) when every proposal was accepted (notation
// paragraph of Section 3; Section 3.1, Eq. (2); Algorithm 1, rejection and
// free-token lines).
//
// Inverse-CDF sampling in target-id order over tiles of 256 ids (8 consecutive
// ids per lane of one warp, so a tile needs shuffles only, no block barrier).
// Values are carried unnormalised: e(t) = exp2((x_t - M)*scale) = p(t)*S and
// r'(t) = max(0, e(t) - q'(t)*S).
//   pass 1  every warp takes a run of tiles of row j = n_b; per tile one coalesced
//           128-bit load of the logits, one coalesced read of the inverse map (the
//           draft id of each target id, -1 outside the map's image), a predicated
//           gather of the drafter's probability for the ids that have one, r' of
//           its eight ids (with the two ids Eq. (2) singles out) and one warp sum:
//           the tile's value. Whole tiles go in pairs, software-pipelined: the
//           inverse-map entries of the next pair are requested before the gathers
//           of the current pair, so a pair costs one memory round trip (the
//           entries of a warp's first pair, like everything else that does not
//           depend on the verification kernels, are requested before the kernel
//           waits for them);
//   ticket  blocks never wait for each other: the block that draws the
//           sequence's last ticket continues alone;
//   pass 2  that block scans the tile values in parallel (total,
//           target = u * total), finds the tile in which the running sum crosses
//           the target, and one warp evaluates r'(t) of that single tile id by id
//           and scans inside it. Without residual mass it draws from p_j (it then
//           redoes the tile sums with e alone).
// A lane adds its eight values in fp32 in index order and a tile's value is the
// fp32 warp sum of the lanes (fixed shuffle tree); sums and scans across tiles,
// and the scan inside the chosen tile, are fp64 in a fixed order: the result is
// reproducible, and the only difference to exact arithmetic is the fp32 rounding
// of the terms and of the tile sums.
//
// Vocabulary shards (the rows split by columns over several GPUs) use the same
// kernel in two further modes. A shard owns a window of whole tiles:
//   mode 1  pass 1 over the window, then the last block adds the window's tile
//           values: the shard's share of the residual mass (and, when that is
//           zero, of the mass of p_j, for the fallback);
//   mode 2  after the shares of all shards were exchanged: every shard forms the
//           same total and target = u * total, finds the shard in which the running
//           sum over shards crosses the target, and that shard alone scans its
//           window (offset by the shares before it) as in pass 2.
#include <float.h>

#include "od_common.cuh"
#include "od_decide.cuh"

namespace {

constexpr int WARPS = OD_SAMPLE_THREADS / 32;
constexpr int EPT = OD_SAMPLE_TILE / 32;                  // ids per lane per tile (8)

// A 16-byte load of logits, which are read once: past L1, whose lines are better spent on the
// drafter's row, which the gathers come back to, and on the inverse map, which the blocks of
// other sequences on the same multiprocessor read too (od_sample_residual 14.7 -> 14.2 us on
// the batched workload; the inverse map past L1 as well: 15.5 us).
__device__ __forceinline__ uint4 ld_once(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
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
    double *tile_val;                   // [B][ntiles] sum over the tile of r'
    unsigned int *ticket;
    // vocabulary shards: this shard's tiles are [tile_lo, tile_hi); `logits` points at
    // its first column (target id col0), v_p is the id one past its last column
    int32_t tile_lo, tile_hi, col0;
    int32_t n_shards, shard_index;
    const double *mass_all;             // [n_shards][B][2] (residual share, share of p_j or 0)
    double *mass_out;                   // [B][2] this shard's shares
    int32_t early;                      // 1: the translation's outputs may be read before griddepcontrol.wait
    // od_step: no decide kernel ran; the decisions of step 2 are taken here, by every block of a
    // sequence alike, from the partials the streaming pass left, and the sequence's block 0
    // writes step 2's outputs (the w_ pointers; row_max, row_sum, n_accepted above are not read)
    StreamPlan plan;
    float *w_row_max, *w_row_sum, *w_p_sel, *w_ratio;
    int32_t *w_n_accepted, *w_n_draft;
    uint32_t *w_vflags;
};

// what one sequence's warps need to evaluate r(t)
struct SeqState {
    const char *row;
    const float *q_row;
    float c, S, scale;      // e(t) = exp2(fma(x_t, scale, -c)); S is the row sum relative to c
    bool residual;
    int32_t ngram_token, prefix_token, first_draft;
    float ngram_prob, prefix_val;
};

// Values are carried UNNORMALISED: with c = fl(M*scale), e(t) = exp2(x_t*scale - c) and
// S = (row sum relative to M) * exp2(M*scale - c), so that p(t) = e(t)/S exactly as
// before but one fused multiply-add per id replaces a subtraction and a product,
//   residual   r'(t) = max(0, e(t) - q'(t)*S) = S * max(0, p(t) - q'(t))
//   free token r'(t) = e(t)
// so one multiplication by 1/S at the very end replaces one per element, and the
// inverse-CDF pick (target = u * sum r') is unchanged by the common factor.
__device__ __forceinline__ float resid_of(const SeqState &q, float x, float qq)
{
    return fmaxf(0.f, fmaf(-qq, q.S, od_ex2(fmaf(x, q.scale, -q.c))));
}

// Eq. (2): the two ids whose q' is not the drafter's row. Only the lane that owns such
// an id (its ids are t0 .. t0 + EPT - 1) redoes it: prefix sub-token first, the n-gram
// token last.
template <int DTYPE>
__device__ __forceinline__ void eq2_ids(const SeqState &q, const SampleArgs &a, int t0, float *r)
{
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

// r'(t) of the EPT consecutive ids this lane owns in `tile`; ids >= v_p give 0
template <int DTYPE>
__device__ __forceinline__ void tile_values(const SeqState &q, const SampleArgs &a, bool residual,
                                            int tile, int lane, float *r)
{
    const int t0 = tile * OD_SAMPLE_TILE + lane * EPT;
    if (t0 + EPT <= a.v_p) {
        float x[EPT];
        if (DTYPE == OD_BF16) {
            const uint4 v = ld_once(q.row + (size_t)t0 * 2);
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
            for (int e = 0; e < EPT; ++e) r[e] = od_ex2(fmaf(x[e], q.scale, -q.c));
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
                    r[e] = od_ex2(fmaf(xv, q.scale, -q.c));
                }
            }
        }
    }
    if (residual) eq2_ids<DTYPE>(q, a, t0, r);
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

// e(t) of the EPT consecutive ids this lane owns in `tile`; ids >= v_p give 0
template <int DTYPE>
__device__ __forceinline__ void tile_e_values(const SeqState &q, const SampleArgs &a, int tile, int lane, float *r)
{
    const int t0 = tile * OD_SAMPLE_TILE + lane * EPT;
    if (t0 + EPT <= a.v_p) {
        float x[EPT];
        if (DTYPE == OD_BF16) {
            const uint4 v = ld_once(q.row + (size_t)t0 * 2);
            x[0] = od_bf16_lo(v.x); x[1] = od_bf16_hi(v.x); x[2] = od_bf16_lo(v.y); x[3] = od_bf16_hi(v.y);
            x[4] = od_bf16_lo(v.z); x[5] = od_bf16_hi(v.z); x[6] = od_bf16_lo(v.w); x[7] = od_bf16_hi(v.w);
        } else {
            const float4 v0 = __ldg((const float4 *)(q.row + (size_t)t0 * 4));
            const float4 v1 = __ldg((const float4 *)(q.row + (size_t)t0 * 4) + 1);
            x[0] = v0.x; x[1] = v0.y; x[2] = v0.z; x[3] = v0.w;
            x[4] = v1.x; x[5] = v1.y; x[6] = v1.z; x[7] = v1.w;
        }
#pragma unroll
        for (int e = 0; e < EPT; ++e) r[e] = od_ex2(fmaf(x[e], q.scale, -q.c));
    } else {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int t = t0 + e;
            r[e] = t < a.v_p ? od_ex2(fmaf(od_load_logit<DTYPE>(q.row, t), q.scale, -q.c)) : 0.f;
        }
    }
}

__device__ __forceinline__ float warp_sum_f32(float v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    return v;
}

// Pass 1, tile by tile (the free token, ragged last tiles, and the fallback of pass 2): every
// id of a tile looks up its draft id in the inverse map (coalesced) and gathers the drafter's
// probability if it has one; NT tiles are in flight per warp.
template <int DTYPE, int NT>
__device__ __forceinline__ void warp_tiles_dense(const SeqState &q, const SampleArgs &a, bool residual, int t_lo,
                                                 int t_hi, int lane, double *tile_val)
{
    for (int t = t_lo; t < t_hi; t += NT) {
        float r[NT][EPT];
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            if (t + i < t_hi) {
                if (residual) tile_values<DTYPE>(q, a, true, t + i, lane, r[i]);
                else tile_e_values<DTYPE>(q, a, t + i, lane, r[i]);
            }
        }
        float mine = 0.f;
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            if (t + i < t_hi) {
                float s = r[i][0];
#pragma unroll
                for (int e = 1; e < EPT; ++e) s += r[i][e];
                s = warp_sum_f32(s);
                if (lane == i) mine = s;
            }
        }
        if (lane < NT && t + lane < t_hi) tile_val[t + lane] = (double)mine;
    }
}

// Inverse-map entries of a warp's first pair of whole tiles [t_lo, t_hi).
__device__ __forceinline__ void first_pair_entries(const SampleArgs &a, int t_lo, int t_hi, int lane, int4 (&ni)[2][2])
{
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int t0 = (t_lo + i < t_hi ? t_lo + i : t_lo) * OD_SAMPLE_TILE + lane * EPT;
        ni[i][0] = __ldg((const int4 *)(a.inv_map + t0));
        ni[i][1] = __ldg((const int4 *)(a.inv_map + t0) + 1);
    }
}

// The same pass for a residual draw, software-pipelined over pairs of WHOLE tiles: the
// inverse-map entries of the next pair are requested before the current pair's gathers,
// so a pair costs one memory round trip, not two. ni: the first pair's entries
// (first_pair_entries), which the caller requested early: they belong to the context and
// depend on nothing the launch in front writes.
template <int DTYPE>
__device__ __forceinline__ void warp_tiles_dense_piped(const SeqState &q, const SampleArgs &a, int t_lo, int t_hi,
                                                       int lane, double *tile_val, int4 (&ni)[2][2])
{
    constexpr int ESZ = DTYPE == OD_BF16 ? 2 : 4;
    for (int t = t_lo; t < t_hi; t += 2) {
        int32_t d[2][EPT];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            d[i][0] = ni[i][0].x; d[i][1] = ni[i][0].y; d[i][2] = ni[i][0].z; d[i][3] = ni[i][0].w;
            d[i][4] = ni[i][1].x; d[i][5] = ni[i][1].y; d[i][6] = ni[i][1].z; d[i][7] = ni[i][1].w;
        }
        if (t + 2 < t_hi) {
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int t0 = (t + 2 + i < t_hi ? t + 2 + i : t + 2) * OD_SAMPLE_TILE + lane * EPT;
                ni[i][0] = __ldg((const int4 *)(a.inv_map + t0));
                ni[i][1] = __ldg((const int4 *)(a.inv_map + t0) + 1);
            }
        }
        const bool two = t + 1 < t_hi;
        uint4 raw[2][DTYPE == OD_BF16 ? 1 : 2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint4 *src = (const uint4 *)(q.row + (size_t)((i == 0 || two ? t + i : t) * OD_SAMPLE_TILE + lane * EPT) * ESZ);
            raw[i][0] = ld_once(src);
            if (DTYPE != OD_BF16) raw[i][1] = ld_once(src + 1);
        }
        float qq[2][EPT];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int e = 0; e < EPT; ++e) qq[i][e] = d[i][e] >= 0 ? __ldg(q.q_row + d[i][e]) : 0.f;
        }
        float mine = 0.f;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            float x[EPT], r[EPT];
            if (DTYPE == OD_BF16) {
                const uint4 v = raw[i][0];
                x[0] = od_bf16_lo(v.x); x[1] = od_bf16_hi(v.x); x[2] = od_bf16_lo(v.y); x[3] = od_bf16_hi(v.y);
                x[4] = od_bf16_lo(v.z); x[5] = od_bf16_hi(v.z); x[6] = od_bf16_lo(v.w); x[7] = od_bf16_hi(v.w);
            } else {
                const uint4 v0 = raw[i][0], v1 = raw[i][DTYPE == OD_BF16 ? 0 : 1];
                x[0] = __uint_as_float(v0.x); x[1] = __uint_as_float(v0.y); x[2] = __uint_as_float(v0.z); x[3] = __uint_as_float(v0.w);
                x[4] = __uint_as_float(v1.x); x[5] = __uint_as_float(v1.y); x[6] = __uint_as_float(v1.z); x[7] = __uint_as_float(v1.w);
            }
#pragma unroll
            for (int e = 0; e < EPT; ++e) r[e] = resid_of(q, x[e], qq[i][e]);
            eq2_ids<DTYPE>(q, a, (t + i) * OD_SAMPLE_TILE + lane * EPT, r);
            float sum = r[0];
#pragma unroll
            for (int e = 1; e < EPT; ++e) sum += r[e];
            sum = warp_sum_f32(sum);
            if (lane == i) mine = sum;
        }
        if (lane < 2 && t + lane < t_hi) tile_val[t + lane] = (double)mine;
    }
}

// Sum of s_val[my_lo, my_hi) over the block's threads in the order of the scan of
// pass 2 (a thread's run, lanes in order, warps in order); every thread gets it.
__device__ __forceinline__ double block_total(const double *s_val, int my_lo, int my_hi, double *s_warp)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double inc = 0.0;
    for (int t = my_lo; t < my_hi; ++t) inc += s_val[t];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double v = __shfl_up_sync(0xFFFFFFFFu, inc, off);
        if (lane >= off) inc += v;
    }
    __syncthreads();                                // s_warp may still be read from an earlier call
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    double tot = 0.0;
    for (int w = 0; w < WARPS; ++w) tot += s_warp[w];
    return tot;
}

// MODE 0: the whole step on full rows; 1: a shard's mass shares; 2: a shard's pick.
// FUSED (mode 0 only): the launch in front is the streaming pass of od_verify itself; its
// decide kernel is folded into this kernel's prologue (see SampleArgs).
template <int DTYPE, int MODE, bool FUSED>
__global__ void __launch_bounds__(OD_SAMPLE_THREADS, 4)
od_sample_kernel(const SampleArgs a)
{
    __shared__ float s_M[FUSED ? OD_MAX_K + 1 : 1], s_S[FUSED ? OD_MAX_K + 1 : 1];
    __shared__ int s_red[2][WARPS];
    __shared__ unsigned int s_vbits;
    extern __shared__ __align__(16) unsigned char s_dyn[];   // ntiles x 8 bytes
    double *s_val = (double *)s_dyn;                         // pass 2: tile values
    __shared__ double s_warp[WARPS];
    __shared__ unsigned int s_last;
    __shared__ int s_tile, s_lastmass, s_token;
    __shared__ double s_before, s_total;
    __shared__ double s_cross[OD_SAMPLE_THREADS];           // pass 2: the sum in front of a thread's crossing tile

    // grid = (sequences, parts of a row): blocks with neighbouring indices, which often end up on
    // one multiprocessor, then work on the same tiles of different sequences and share the
    // inverse-map entries in L1
    const int b = blockIdx.x;
    const unsigned int part = blockIdx.y, nparts = gridDim.y;
    const int K = a.K_max;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // Under programmatic dependent launch this grid is resident while the verification
    // kernels still run. What the translation kernel wrote (it finished before them) is
    // read now, for every position the step can stop at: lane k of every warp prepares
    // position k. After the wait only n_accepted and the row statistics are missing.
    // (a.early = 0: the launch before this one was not od_verify; everything waits.)
    asm volatile("griddepcontrol.launch_dependents;");
    if (!a.early) asm volatile("griddepcontrol.wait;" ::: "memory");
    // Two memory round trips, not a chain of four: everything that is addressed by (b, lane)
    // alone is requested at once, whether or not it will be used (lane < K keeps the
    // addresses inside the arrays); what is addressed by those values comes second.
    int mb = a.m[b];
    const bool stop = a.tail_kind[b] == OD_TAIL_UNMAPPED_STOP;
    const float T = a.temperature[b];
    int32_t l_s0 = 0, l_len = 1, l_tgt = -1, l_did = -1;
    float l_qp = 0.f;
    if (lane < K) {
        const size_t o = (size_t)b * K + lane;
        l_s0 = a.span_start[o];
        l_len = a.span_len[o];
        l_tgt = a.tgt_ids[o];
        l_qp = a.q_prime[o];
        l_did = a.draft_ids[o];
    }
    mb = mb < 0 ? 0 : (mb > K ? K : mb);
    int32_t e_s0 = 0, e_len = 1, e_tgt = -1, e_d1 = -1, e_pm = -1;
    float e_qp = 0.f, e_qd1 = 0.f;
    {
        const bool live = lane < K && lane <= mb;
        if (live) {
            e_s0 = l_s0 < 0 ? 0 : (l_s0 >= K ? K - 1 : l_s0);
            e_len = lane < mb ? l_len : 1;
        }
        const int32_t d1 = __shfl_sync(0xFFFFFFFFu, l_did, e_s0);   // the span's first draft token
        if (live && e_len >= 2) {
            e_tgt = l_tgt;
            e_qp = l_qp;
            if (d1 >= 0 && d1 < a.v_q) {
                e_d1 = d1;
                e_pm = __ldg(a.vocab_map + d1);
                e_qd1 = __ldg(a.q_rows + ((size_t)b * K + e_s0) * a.v_q + d1);
            }
        }
    }

    // FUSED, still before the wait: where the rows' partials will be (sums of m), and position
    // k's inputs of the acceptance test in lane k
    int before = 0, total = 0;
    float d_xt = 0.f, d_q = 0.f, d_u = 0.f;
    bool d_tok = false;
    int32_t d_span = 0;
    if (FUSED) {
        for (int i = threadIdx.x; i < a.B; i += OD_SAMPLE_THREADS) {
            const int v = clamp_m(a.m[i], K);
            total += v;
            if (i < b) before += v;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            before += __shfl_xor_sync(0xFFFFFFFFu, before, off);
            total += __shfl_xor_sync(0xFFFFFFFFu, total, off);
        }
        if (lane == 0) { s_red[0][warp] = before; s_red[1][warp] = total; }
        if (threadIdx.x == 0) s_vbits = 0;
        if (lane < mb) {
            const int32_t t = l_tgt;
            d_tok = t >= 0 && t < a.v_p;
            const char *row_k = (const char *)a.logits +
                                ((size_t)b * a.seq_stride + (size_t)lane * a.row_stride) * (DTYPE == OD_BF16 ? 2 : 4);
            if (d_tok) d_xt = od_load_logit<DTYPE>(row_k, t);
            d_q = l_qp;
            d_u = od_uniform(a.seed[b], a.step, (uint32_t)lane, 0u);
            d_span = l_len;
        }
        __syncthreads();
        before = 0; total = 0;
        for (int w = 0; w < WARPS; ++w) { before += s_red[0][w]; total += s_red[1][w]; }
    }

    // a shard's tiles and ids keep their numbers of the full row
    const int tile_lo = MODE == 0 ? 0 : a.tile_lo;
    const int tile_hi = MODE == 0 ? a.ntiles : a.tile_hi;
    // pass 1's whole tiles of this warp, and the inverse-map entries of their first pair
    const int p_lo = tile_lo + ((int)part * WARPS + warp) * a.tiles_per_warp;
    int p_hi = p_lo + a.tiles_per_warp;
    if (p_hi > tile_hi) p_hi = tile_hi;
    const int p_hi_w = p_hi < a.v_p / OD_SAMPLE_TILE ? p_hi : a.v_p / OD_SAMPLE_TILE;
    int4 ni[2][2] = {};
    if (MODE != 2 && p_lo < p_hi_w) first_pair_entries(a, p_lo, p_hi_w, lane, ni);

    // n_accepted and the row statistics come from the verification kernels
    if (a.early) asm volatile("griddepcontrol.wait;" ::: "memory");

    int fused_n = 0;
    if (FUSED) {
        // ---- step 2's decisions (what od_verify_decide_kernel does, same arithmetic, same order)
        const bool bad_T = !(T > 0.f);
        const float dscale = bad_T ? 0.f : 1.4426950408889634f / T;
        for (int r = warp; r <= mb; r += WARPS) {
            const int row_slot = b * (K + 1) + r;
            float c, sum, mx;
            merge_row_partials(a.plan, row_slot, row_partial_segments(a.plan, b, r, before, total), lane, c, sum, mx);
            if (lane == 0) {
                const float S = row_sum_of(c, sum, mx, dscale);
                s_M[r] = mx; s_S[r] = S;
                if (part == 0) { a.w_row_max[row_slot] = mx; a.w_row_sum[row_slot] = S; }
                if (!(S > 0.f) || !(S <= FLT_MAX)) atomicOr(&s_vbits, 1u);
            }
        }
        __syncthreads();
        // every warp takes the decisions for itself (lane k = position k holds the inputs in
        // every warp): no second barrier; warp 0 of the sequence's first block stores them
        int n = 0;
        {
            bool acc = false, bnd = false;
            Acceptance d = {};
            if (lane < mb) {
                d = accept_position(s_M[lane], s_S[lane], dscale, d_tok, d_xt, d_q, d_u);
                acc = d.accept; bnd = d.boundary;
            }
            const unsigned int accmask = __ballot_sync(0xFFFFFFFFu, acc);
            while (n < mb && (accmask >> n & 1u)) ++n;
            if (bad_T) n = 0;
            if (part == 0 && warp == 0) {
                if (lane < mb) { a.w_p_sel[(size_t)b * K + lane] = d.p; a.w_ratio[(size_t)b * K + lane] = d.ratio; }
                const unsigned int bndmask = __ballot_sync(0xFFFFFFFFu, bnd);
                int nd = lane < n ? d_span : 0;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) nd += __shfl_xor_sync(0xFFFFFFFFu, nd, off);
                if (lane == 0) {
                    uint32_t f = bndmask & OD_VF_BOUNDARY_MASK;
                    if (s_vbits & 1u) f |= OD_VF_NONFINITE;
                    if (bad_T) f |= OD_VF_BAD_TEMPERATURE;
                    a.w_n_accepted[b] = n; a.w_n_draft[b] = nd; a.w_vflags[b] = f;
                }
            }
        }
        fused_n = n;
    }

    if (!(T > 0.f)) {                              // every block of the sequence leaves here
        if (part == 0 && threadIdx.x == 0) {
            if (MODE == 1) {
                a.mass_out[2 * b] = 0.0; a.mass_out[2 * b + 1] = 0.0;
            } else {
                a.out_token[b] = -1; a.resid_mass[b] = 0.f; a.flags[b] = OD_SF_BAD_TEMPERATURE;
            }
        }
        return;
    }
    float rm = 0.f, rs = 0.f;                      // lane k: statistics of row k
    if (lane <= mb) {
        rm = FUSED ? s_M[lane] : a.row_max[b * (K + 1) + lane];
        rs = FUSED ? s_S[lane] : a.row_sum[b * (K + 1) + lane];
    }
    int j = FUSED ? fused_n : a.n_accepted[b];
    j = j < 0 ? 0 : (j > mb ? mb : j);
    const size_t esz = DTYPE == OD_BF16 ? 2 : 4;
    // a shard's row pointer is moved back by the shard's first column, and only ids of
    // the window are read
    SeqState q;
    q.row = (const char *)a.logits + ((size_t)b * a.seq_stride + (size_t)j * a.row_stride) * esz;
    if (MODE != 0) q.row -= (size_t)a.col0 * esz;
    q.scale = 1.4426950408889634f / T;
    {
        // reference exponent c = fl(M*scale); the rounding of c goes into S exactly:
        // sum_t exp2(x_t*scale - c) = (sum_t exp2((x_t - M)*scale)) * exp2(M*scale - c)
        const float M = __shfl_sync(0xFFFFFFFFu, rm, j);
        q.c = fmaxf(M * q.scale, -FLT_MAX);
        q.S = __shfl_sync(0xFFFFFFFFu, rs, j) * od_ex2(fmaf(M, q.scale, -q.c));
    }
    q.residual = (j < mb) || stop;
    q.ngram_token = -1; q.prefix_token = -1; q.first_draft = -1; q.ngram_prob = 0.f; q.prefix_val = 0.f;
    q.q_row = a.q_rows;
    {
        // position j's preparation (j < K whenever the draw is a residual one)
        const int src = j < K ? j : 0;
        const int32_t s0 = __shfl_sync(0xFFFFFFFFu, e_s0, src), len = __shfl_sync(0xFFFFFFFFu, e_len, src);
        const int32_t tgt = __shfl_sync(0xFFFFFFFFu, e_tgt, src), d1 = __shfl_sync(0xFFFFFFFFu, e_d1, src);
        const int32_t pm = __shfl_sync(0xFFFFFFFFu, e_pm, src);
        const float qp = __shfl_sync(0xFFFFFFFFu, e_qp, src), qd1 = __shfl_sync(0xFFFFFFFFu, e_qd1, src);
        if (q.residual) {
            q.q_row = a.q_rows + ((size_t)b * K + s0) * a.v_q;
            // the gathers of pass 1 come two round trips from now: have the copy engine pull
            // this block's share of the drafter's row into L2 meanwhile
            if (MODE != 2 && threadIdx.x == 0) {
                const size_t row_bytes = (size_t)a.v_q * 4 / 16 * 16;
                size_t lo = (row_bytes / nparts * part) / 16 * 16;
                size_t hi = part + 1 == nparts ? row_bytes : (row_bytes / nparts * (part + 1)) / 16 * 16;
                const char *base = (const char *)q.q_row;
                if (((uintptr_t)base & 15u) == 0 && hi > lo)
                    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(base + lo), "r"((uint32_t)(hi - lo)) : "memory");
            }
            if (len >= 2) {
                q.ngram_token = tgt;
                q.ngram_prob = qp;
                if (d1 >= 0) {
                    q.first_draft = d1;
                    q.prefix_token = pm;
                    q.prefix_val = qd1 - q.ngram_prob;
                }
            }
        }
    }

    const int ntiles = a.ntiles;
    double *tile_val = a.tile_val + (size_t)b * ntiles;

    if (MODE != 2) {
        // ---- pass 1: the value of every tile ----
        {
            const int t_lo = p_lo, t_hi = p_hi;
            if (t_lo < t_hi) {
                // whole tiles pipelined; the row's ragged last tile (if it is this warp's) on its own
                const int hi_w = p_hi_w;
                if (q.residual) {
                    if (t_lo < hi_w) warp_tiles_dense_piped<DTYPE>(q, a, t_lo, hi_w, lane, tile_val, ni);
                    if (hi_w < t_hi) warp_tiles_dense<DTYPE, 2>(q, a, true, hi_w > t_lo ? hi_w : t_lo, t_hi, lane, tile_val);
                } else {
                    warp_tiles_dense<DTYPE, 2>(q, a, false, t_lo, t_hi, lane, tile_val);
                }
            }
        }
        // The tile values are read by another block: the barrier orders this block's stores
        // before thread 0's fence, the fence before its ticket (release); the block that
        // draws the last ticket fences again before anyone in it reads (acquire).
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            s_last = atomicAdd(a.ticket + b, 1u) == nparts - 1 ? 1u : 0u;
            __threadfence();
        }
        __syncthreads();
        if (!s_last) return;
    }

    // ---- pass 2 (one block per sequence) ----
    bool residual = q.residual;
    uint32_t flags = residual ? 0u : OD_SF_BONUS;
    const int per = (tile_hi - tile_lo + OD_SAMPLE_THREADS - 1) / OD_SAMPLE_THREADS;
    const int my_lo = tile_lo + threadIdx.x * per < tile_hi ? tile_lo + threadIdx.x * per : tile_hi;
    const int my_hi = my_lo + per < tile_hi ? my_lo + per : tile_hi;
    // tile values (rounding can leave a tile without residual mass slightly negative): four
    // requests per thread at a time, and the draw's uniform worked out while they travel
    float u = 0.f;
    const uint64_t seed_b = MODE == 1 ? 0ull : a.seed[b];   // requested with the tile values, used behind them
    for (int t0 = tile_lo + threadIdx.x, first = 1; first || t0 < tile_hi; t0 += 4 * OD_SAMPLE_THREADS, first = 0) {
        double v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = t0 + i * OD_SAMPLE_THREADS;
            v[i] = t < tile_hi ? __ldcg(tile_val + t) : 0.0;
        }
        if (MODE != 1 && first) u = od_uniform(seed_b, a.step, (uint32_t)j, 1u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = t0 + i * OD_SAMPLE_THREADS;
            if (t < tile_hi) s_val[t] = fmax(0.0, v[i]);
        }
    }
    if (MODE != 2 && threadIdx.x == 0) a.ticket[b] = 0;
    __syncthreads();

    if (MODE == 1) {
        // ---- this shard's shares ----
        const double mass_r = block_total(s_val, my_lo, my_hi, s_warp);
        double mass_e = 0.0;
        if (residual && !(mass_r > 0.0)) {
            // no residual mass here: should no shard have any, the draw is from p_j
            for (int t_lo = tile_lo + warp * 2; t_lo < tile_hi; t_lo += WARPS * 2)
                warp_tiles_dense<DTYPE, 2>(q, a, false, t_lo, t_lo + 2 < tile_hi ? t_lo + 2 : tile_hi, lane, tile_val);
            __syncthreads();
            for (int t = tile_lo + threadIdx.x; t < tile_hi; t += OD_SAMPLE_THREADS) s_val[t] = fmax(0.0, tile_val[t]);
            __syncthreads();
            mass_e = block_total(s_val, my_lo, my_hi, s_warp);
        }
        if (threadIdx.x == 0) { a.mass_out[2 * b] = mass_r; a.mass_out[2 * b + 1] = mass_e; }
        return;
    }

    double shard_before = 0.0, shard_total = 0.0;      // MODE 2: sums over the shards before this one / all
    if (MODE == 2) {
        double tot_r = 0.0, tot_e = 0.0;
        for (int s = 0; s < a.n_shards; ++s) {
            tot_r += a.mass_all[((size_t)s * a.B + b) * 2];
            tot_e += a.mass_all[((size_t)s * a.B + b) * 2 + 1];
        }
        const bool use_e = residual && !(tot_r > 0.0);
        if (use_e) { residual = false; flags |= OD_SF_ZERO_MASS; }   // the tile values then hold p_j's
        shard_total = use_e ? tot_e : tot_r;
        // the shard in which the running sum crosses the target (else the last one with mass)
        int owner = -1;
        if (shard_total > 0.0) {
            const double target = (double)u * shard_total;
            double c = 0.0;
            int last = -1;
            for (int s = 0; s < a.n_shards; ++s) {
                const double v = a.mass_all[((size_t)s * a.B + b) * 2 + (use_e ? 1 : 0)];
                if (s == a.shard_index) shard_before = c;
                if (v > 0.0) last = s;
                if (c + v > target) { owner = s; break; }
                c += v;
            }
            if (owner < 0) owner = last;
        }
        if (owner != a.shard_index) {
            if (threadIdx.x == 0) {
                const bool report = owner < 0 && a.shard_index == 0;   // no mass anywhere: shard 0 says so
                a.out_token[b] = -1;
                a.resid_mass[b] = report ? (float)(shard_total / (double)q.S) : 0.f;
                a.flags[b] = report ? (flags | OD_SF_ZERO_MASS) : 0u;
            }
            return;
        }
    }

    for (int attempt = 0; attempt < 2; ++attempt) {
        // exclusive scan of the tile values: thread i owns `per` consecutive tiles
        double loc = 0.0;
        for (int t = my_lo; t < my_hi; ++t) loc += s_val[t];
        double inc = loc;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double v = __shfl_up_sync(0xFFFFFFFFu, inc, off);
            if (lane >= off) inc += v;
        }
        if (lane == 31) s_warp[warp] = inc;
        if (threadIdx.x == 0) { s_tile = 0x7FFFFFFF; s_lastmass = -1; s_token = -2; }
        __syncthreads();
        // every thread adds the warps' sums up itself (the same order everywhere): no barrier
        // for the total
        double base = MODE == 2 ? shard_before : 0.0, tot = 0.0;
        for (int w = 0; w < WARPS; ++w) {
            if (w == warp) base += tot;
            tot += s_warp[w];
        }
        if (threadIdx.x == 0) s_total = tot;
        const double Rn = MODE == 2 ? shard_total : tot;   // unnormalised total
        double target = 0.0;
        if (Rn > 0.0) {
            target = (double)u * Rn;
            double c = base + inc - loc;
            int last = -1;
            for (int t = my_lo; t < my_hi; ++t) {
                const double v = s_val[t];
                if (v > 0.0) last = t;
                if (c + v > target) {
                    // first crossing of this run: the tile, and with it who found it, so that
                    // the sum before the tile needs no barrier of its own
                    s_cross[threadIdx.x] = c;
                    atomicMin(&s_tile, t * OD_SAMPLE_THREADS + (int)threadIdx.x);
                    break;
                }
                c += v;
            }
            if (last >= 0) atomicMax(&s_lastmass, last);
        }
        __syncthreads();
        // cumulative sums never decrease, so the smallest reported tile is the crossing;
        // if rounding hid it, take the last tile that has mass
        int t_pick = -1;
        if (Rn > 0.0) {
            if (s_tile != 0x7FFFFFFF) {
                t_pick = s_tile / OD_SAMPLE_THREADS;
                if (threadIdx.x < 32) s_before = s_cross[s_tile % OD_SAMPLE_THREADS];   // warp 0 reads it back below
                __syncwarp();
            } else {
                t_pick = s_lastmass;
                if (t_pick >= my_lo && t_pick < my_hi) {    // its owner publishes the sum before it
                    double c = base + inc - loc;
                    for (int t = my_lo; t < t_pick; ++t) c += s_val[t];
                    s_before = c;
                }
                __syncthreads();                            // (block-uniform: s_tile is the same for all)
            }
        }
        if (t_pick >= 0 && warp == 0) {
            // ---- warp 0 evaluates the chosen tile id by id and scans inside it ----
            float r[EPT];
            if (residual) tile_values<DTYPE>(q, a, true, t_pick, lane, r);
            else tile_e_values<DTYPE>(q, a, t_pick, lane, r);
            const double mine = lane_sum(r);
            double incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const double v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += v;
            }
            const double lbase = s_before + (incl - mine);   // sum before this lane's first id
            const int t0 = t_pick * OD_SAMPLE_TILE + lane * EPT;
            int my_pick = 0x7FFFFFFF, my_last = -1;
            double lo = 0.0, hi = 0.0, c = lbase;
            float run = 0.f;                        // same fp32 order as lane_sum
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
                run = e == 0 ? r[0] : run + r[e];
                const double nc = lbase + (double)run;
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
            const float R = (float)(Rn / (double)q.S);     // residual mass (1 for the free token)
            if (pick != 0x7FFFFFFF) {
                if (my_pick == pick) {              // exactly one lane owns the picked id
                    uint32_t f = flags;
                    if (fmin(target - lo, hi - target) <= OD_TAU_SAMPLE * Rn) f |= OD_SF_BOUNDARY;
                    a.out_token[b] = pick; a.resid_mass[b] = R; a.flags[b] = f;
                    s_token = pick;
                }
            } else if (last >= 0) {
                // rounding: the target lies beyond the tile's last edge
                if (lane == 0) {
                    a.out_token[b] = last; a.resid_mass[b] = R; a.flags[b] = flags | OD_SF_BOUNDARY;
                    s_token = last;
                }
            }                                       // else: the tile holds no mass after all
        }
        __syncthreads();
        if (s_token >= 0) return;
        if (MODE == 2 || !residual || attempt == 1) break;
        // no usable residual mass: draw from p_j instead (rare; this block redoes the row)
        residual = false;
        flags |= OD_SF_ZERO_MASS;
        for (int t_lo = warp * 2; t_lo < ntiles; t_lo += WARPS * 2)
            warp_tiles_dense<DTYPE, 2>(q, a, false, t_lo, t_lo + 2 < ntiles ? t_lo + 2 : ntiles, lane, tile_val);
        __syncthreads();
        for (int t = threadIdx.x; t < ntiles; t += OD_SAMPLE_THREADS) s_val[t] = fmax(0.0, tile_val[t]);
        __syncthreads();
    }
    if (threadIdx.x == 0) {                         // no mass at all (non-finite input)
        a.out_token[b] = -1;
        a.resid_mass[b] = (float)((MODE == 2 ? shard_total : s_total) / (double)q.S);
        a.flags[b] = flags | OD_SF_ZERO_MASS;
    }
}

}  // namespace

// Dynamic shared memory of the kernel for rows of `ntiles` tiles: the tile values of pass 2.
size_t od_sample_smem_bytes(int32_t ntiles) { return (size_t)ntiles * 8; }

// Rows beyond 6144 tiles need more dynamic shared memory than a kernel gets by default: opt
// in (the device must be current; allocates nothing).
cudaError_t od_sample_prepare_device(size_t bytes)
{
    if (bytes <= 48 * 1024) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    const int n = (int)bytes;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_BF16, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_F32, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_BF16, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_F32, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_BF16, 1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_F32, 1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_BF16, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(od_sample_kernel<OD_F32, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, n);
    return e;
}

// mode 0: od_sample_residual; 1 / 2: the two calls of a vocabulary shard
static cudaError_t launch_sample(od_ctx *c, int mode, int32_t B, int32_t K_max, const void *logits,
                                 int32_t dtype, int64_t row_stride, int64_t seq_stride,
                                 const float *row_max, const float *row_sum, const float *q_rows,
                                 const int32_t *draft_ids, const int32_t *tgt_ids,
                                 const float *q_prime, const int32_t *span_start,
                                 const int32_t *span_len, const int32_t *m,
                                 const uint8_t *tail_kind, const int32_t *n_accepted,
                                 const float *temperature, const uint64_t *seed, uint64_t step,
                                 int32_t *out_token, float *resid_mass, uint32_t *flags,
                                 int32_t shard_lo, int32_t shard_len, int32_t n_shards, int32_t shard_index,
                                 const double *mass_all, double *mass_out, cudaStream_t s,
                                 const od_fused_verify *fuse = nullptr)
{
    if (B == 0) return cudaSuccess;
    const int ntiles = c->tiles_per_row;
    const int tile_lo = mode == 0 ? 0 : shard_lo / OD_SAMPLE_TILE;
    const int tile_hi = mode == 0 ? ntiles : (shard_lo + shard_len + OD_SAMPLE_TILE - 1) / OD_SAMPLE_TILE;
    const int wtiles = tile_hi - tile_lo;
    int64_t tpw = c->opt_sample_tiles_per_warp;
    if (tpw <= 0) {
        // one resident wave (four 256-thread blocks per SM) over the whole batch
        const int64_t want = (int64_t)c->sm_count * 4;
        int64_t per_row = want / B;
        if (per_row < 1) per_row = 1;
        tpw = (wtiles + per_row * WARPS - 1) / (per_row * WARPS);
        if (tpw < 1) tpw = 1;
    }
    const int64_t tiles_per_block = tpw * WARPS;
    const int blocks_x = mode == 2 ? 1 : (int)((wtiles + tiles_per_block - 1) / tiles_per_block);
    SampleArgs a = {};
    a.logits = logits; a.row_stride = row_stride; a.seq_stride = seq_stride;
    a.B = B; a.K_max = K_max; a.v_p = mode == 0 ? c->v_p : shard_lo + shard_len; a.v_q = c->v_q;
    a.ntiles = ntiles; a.tiles_per_warp = (int32_t)tpw;
    a.row_max = row_max; a.row_sum = row_sum; a.q_rows = q_rows;
    a.draft_ids = draft_ids; a.tgt_ids = tgt_ids; a.q_prime = q_prime;
    a.span_start = span_start; a.span_len = span_len; a.m = m; a.tail_kind = tail_kind;
    a.n_accepted = n_accepted; a.temperature = temperature; a.seed = seed; a.step = step;
    a.vocab_map = c->d_vocab_map; a.inv_map = c->d_inv_map;
    a.out_token = out_token; a.resid_mass = resid_mass; a.flags = flags;
    a.tile_val = c->d_tile_sums; a.ticket = c->d_samp_ticket;
    a.tile_lo = tile_lo; a.tile_hi = tile_hi; a.col0 = mode == 0 ? 0 : shard_lo;
    a.n_shards = n_shards; a.shard_index = shard_index; a.mass_all = mass_all; a.mass_out = mass_out;
    // the translation kernel releases its successor before it has written anything: directly
    // after it, nothing may be read early
    a.early = c->last_was_map ? 0 : 1;
    if (fuse) {
        a.plan.W = fuse->W; a.plan.n_chunks = fuse->n_chunks; a.plan.span_min = fuse->span_min;
        a.plan.span_a = fuse->span_a; a.plan.seg_warps = fuse->seg_warps; a.plan.partials = c->d_partials;
        a.w_row_max = fuse->row_max; a.w_row_sum = fuse->row_sum; a.w_p_sel = fuse->p_sel; a.w_ratio = fuse->ratio;
        a.w_n_accepted = fuse->n_accepted; a.w_n_draft = fuse->n_draft_accepted; a.w_vflags = fuse->flags;
    }
    c->last_was_map = false;
    if (mode != 2) {
        c->info[2] = (int64_t)blocks_x * B;
        c->info[3] = tpw;
    }

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)B, (unsigned)blocks_x);
    cfg.blockDim = dim3(OD_SAMPLE_THREADS);
    cfg.dynamicSmemBytes = od_sample_smem_bytes(ntiles);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->opt_pdl ? 1 : 0;
    const bool bf = dtype == OD_BF16;
    if (mode == 0 && fuse)
        return bf ? cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_BF16, 0, true>, a)
                  : cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_F32, 0, true>, a);
    if (mode == 0)
        return bf ? cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_BF16, 0, false>, a)
                  : cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_F32, 0, false>, a);
    if (mode == 1)
        return bf ? cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_BF16, 1, false>, a)
                  : cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_F32, 1, false>, a);
    return bf ? cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_BF16, 2, false>, a)
              : cudaLaunchKernelEx(&cfg, od_sample_kernel<OD_F32, 2, false>, a);
}

cudaError_t od_launch_sample(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                             int32_t dtype, int64_t row_stride, int64_t seq_stride,
                             const float *row_max, const float *row_sum, const float *q_rows,
                             const int32_t *draft_ids, const int32_t *tgt_ids,
                             const float *q_prime, const int32_t *span_start,
                             const int32_t *span_len, const int32_t *m,
                             const uint8_t *tail_kind, const int32_t *n_accepted,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             int32_t *out_token, float *resid_mass, uint32_t *flags,
                             cudaStream_t s, const od_fused_verify *fuse)
{
    return launch_sample(c, 0, B, K_max, logits, dtype, row_stride, seq_stride, row_max, row_sum, q_rows,
                         draft_ids, tgt_ids, q_prime, span_start, span_len, m, tail_kind, n_accepted,
                         temperature, seed, step, out_token, resid_mass, flags, 0, 0, 1, 0, nullptr, nullptr, s,
                         fuse);
}

cudaError_t od_launch_sample_shard_mass(od_ctx *c, int32_t B, int32_t K_max, int32_t shard_lo,
                                        int32_t shard_len, const void *logits, int32_t dtype,
                                        int64_t row_stride, int64_t seq_stride, const float *row_max,
                                        const float *row_sum, const float *q_rows, const int32_t *draft_ids,
                                        const int32_t *tgt_ids, const float *q_prime,
                                        const int32_t *span_start, const int32_t *span_len, const int32_t *m,
                                        const uint8_t *tail_kind, const int32_t *n_accepted,
                                        const float *temperature, double *mass, cudaStream_t s)
{
    return launch_sample(c, 1, B, K_max, logits, dtype, row_stride, seq_stride, row_max, row_sum, q_rows,
                         draft_ids, tgt_ids, q_prime, span_start, span_len, m, tail_kind, n_accepted,
                         temperature, nullptr, 0, nullptr, nullptr, nullptr, shard_lo, shard_len, 1, 0,
                         nullptr, mass, s);
}

cudaError_t od_launch_sample_shard_pick(od_ctx *c, int32_t B, int32_t K_max, int32_t n_shards,
                                        int32_t shard_index, int32_t shard_lo, int32_t shard_len,
                                        const double *mass_all, const void *logits, int32_t dtype,
                                        int64_t row_stride, int64_t seq_stride, const float *row_max,
                                        const float *row_sum, const float *q_rows, const int32_t *draft_ids,
                                        const int32_t *tgt_ids, const float *q_prime,
                                        const int32_t *span_start, const int32_t *span_len, const int32_t *m,
                                        const uint8_t *tail_kind, const int32_t *n_accepted,
                                        const float *temperature, const uint64_t *seed, uint64_t step,
                                        int32_t *out_token, float *resid_mass, uint32_t *flags, cudaStream_t s)
{
    return launch_sample(c, 2, B, K_max, logits, dtype, row_stride, seq_stride, row_max, row_sum, q_rows,
                         draft_ids, tgt_ids, q_prime, span_start, span_len, m, tail_kind, n_accepted,
                         temperature, seed, step, out_token, resid_mass, flags, shard_lo, shard_len, n_shards,
                         shard_index, mass_all, nullptr, s);
}
