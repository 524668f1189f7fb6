// Step 2: temperature softmax statistics of the m_b + 1 target-logit rows,
// acceptance ratios and the accepted prefix (Algorithm 1, target-probability
// and rejection-sampling lines; acceptance ratio of Section 3.1).
//
// Two launches.
//
// (1) od_verify_stream_kernel: one streaming pass in which every logit crosses
// HBM exactly once (128-bit loads, four in flight per thread, one resident wave of
// 32 warps per SM: two blocks of 16 warps for rows of 128 KB and more, four blocks
// of 8 warps for shorter rows). The bytes are split evenly over the
// blocks, whatever the mix of row counts. The unit of work is 512 contiguous
// bytes of a row; a row has W units; the rows to read are laid end to end in
// two flat index spaces and every block takes one contiguous span of each:
//   space A  row 0 of every sequence. It is always read and its split needs
//            nothing from the device, so when the library knows that the
//            logits are complete (see `a_early`) a block works through its
//            span before it waits for the launch in front (programmatic
//            dependent launch): the translation kernel, or the previous
//            launch's decide kernel, is hidden behind useful traffic;
//   space B  rows 1..m_b, split by the prefix sums of m, which every warp
//            works out for itself (at most 2048 sequences per launch).
// A span is cut at row ends into segments; every warp of the block reduces its
// share of a segment to one partial (reference exponent c, sum of
// exp2(x*scale - c), exact maximum) and stores it. No atomics, no fences, no
// barriers in the stream: no warp waits for another.
//
// (2) od_verify_decide_kernel: one block per sequence, one warp per row. Before
// it waits for the stream kernel it loads what does not depend on it (m, T,
// t_i, q'(t_i), x[t_i], the Philox uniforms); afterwards warp r merges the
// partials of row r, evaluates p(t_i), the ratio and the accept bit, and thread
// 0 turns the bits into the accepted prefix.
//
// Arithmetic: exp((x - M)/T) is evaluated as exp2(fma(x, s, -c)) with
// s = log2(e)/T and c = fl(r*s) for a running reference r >= every element
// absorbed so far (refreshed once per group of vectors, not per element). A
// partial is carried relative to its own c, partials are merged in the scaled
// domain, and the row sum relative to the exact maximum M is recovered at the
// end as S_c * exp2(fma(-M, s, c)), which removes the rounding of c. M itself
// is tracked separately (packed bf16x2 maxima for bf16 rows). The reduction
// order is fixed by (m, grid): results are bit-identical from run to run.
//
// Vocabulary-sharded variant (the target's output layer split by columns over
// several GPUs): a shard streams its own columns with the same stream kernel,
// od_verify_shard_stats_kernel folds the partials of a row into one record
// (c, sum, max, x[t_i] if the shard owns t_i), the records of all shards are
// exchanged by the caller, and od_verify_finish_kernel merges them (the same
// pair algebra) and takes the decisions of the decide kernel.
#include <float.h>

#include "od_common.cuh"
#include "od_decide.cuh"

namespace {

// Two block shapes of the stream kernel. Rows of 128 KB and more (256 units) go to blocks of
// 16 warps, two per multiprocessor: fewer blocks of different age share a multiprocessor,
// and od_verify is 0.5 us (batched 128256-id rows) to 8 us (512 x 9 rows of 152064 ids)
// faster; shorter rows would leave a warp of such a block less than two groups of loads per
// row, and keep blocks of 8 warps, four per multiprocessor. The template parameter TW is
// the number of warps; a block segment has TW partials.
constexpr int NARROW_WARPS = 8, WIDE_WARPS = 16;
constexpr int WIDE_MIN_UNITS = 256;
static_assert(OD_VERIFY_SEG_MAX % WIDE_WARPS == 0 && OD_VERIFY_SEG_MAX / WIDE_WARPS >= 3, "segments per row");
constexpr int U = 4;                            // 16-byte loads in flight per thread
constexpr int A_PARK = 8;                       // partials of space A a block can hold back
#ifndef OD_VERIFY_MAXNREG
#define OD_VERIFY_MAXNREG 56
#endif
#ifndef OD_VERIFY_BLOCKS_PER_SM
#define OD_VERIFY_BLOCKS_PER_SM 4               // resident blocks per SM the register budget allows
#endif

struct VerifyArgs {
    const void *logits;
    int64_t row_stride, seq_stride;     // elements
    int32_t B, K_max, v_p;
    int32_t W;                          // 512-byte units per row
    int32_t n_chunks;                   // blocks of the stream grid
    int32_t seg_warps;                  // warps of a block = partials of a block segment (8 or 16)
    int32_t span_min;                   // keeps a row within OD_VERIFY_SEG_MAX / seg_warps block segments
    int32_t span_a;                     // units of space A per block
    int32_t a_early;                    // 1: space A is streamed before griddepcontrol.wait (the caller allows
                                        // it and a block's span of space A has at most A_PARK segments)
    uint32_t w_mul, w_sh;               // n / W and n / n_chunks for n < 2^31 by multiplication (fast_div)
    uint32_t c_mul, c_sh;
    const int32_t *tgt_ids;
    const float *q_prime;
    const int32_t *span_len;
    const int32_t *m;
    const float *temperature;
    const uint64_t *seed;
    uint64_t step;
    float *row_max, *row_sum, *p_sel, *ratio;
    int32_t *n_accepted, *n_draft_accepted;
    uint32_t *flags;
    float4 *partials;                   // [row slot][OD_VERIFY_SEG_MAX] (c, sum, max, -)
    // vocabulary shards: v_p above is then the number of columns of this shard
    int32_t col0;                       // target id of the shard's first column
    int32_t n_shards;
    float4 *stats;                      // [row slot] (c, sum, max, x[t_i] or -inf) of this shard
    const float4 *stats_all;            // [n_shards][rows][4], rows = batch * (K_max + 1)
    int64_t stats_rows;
};

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Running state of one thread inside a segment.
template <int DTYPE>
struct Lane {
    float c, s;             // reference exponent (scaled domain), sum of exp2(x*scale - c)
    float mx;               // fp32 rows: running maximum
    uint32_t pm;            // bf16 rows: packed running maxima (exact)
    __device__ __forceinline__ void reset()
    {
        c = -FLT_MAX; s = 0.f; mx = -INFINITY; pm = 0xFF80FF80u;
    }
    // make c >= gm*scale (branch-free: one rescale per group of vectors)
    __device__ __forceinline__ void raise(float gm, float scale)
    {
        const float cn = fmaxf(fmaxf(gm * scale, -FLT_MAX), c);
        s *= od_ex2(c - cn);
        c = cn;
    }
    __device__ __forceinline__ float max_seen() const
    {
        if (DTYPE == OD_BF16) return fmaxf(od_bf16_lo(pm), od_bf16_hi(pm));
        return mx;
    }
};

// absorb N 16-byte vectors held in registers
template <int DTYPE, int N>
__device__ __forceinline__ void absorb(Lane<DTYPE> &L, const uint4 *v, float scale)
{
    if (DTYPE == OD_BF16) {
        uint32_t g = L.pm;
#pragma unroll
        for (int u = 0; u < N; ++u) {
            g = bf16x2_max(g, v[u].x); g = bf16x2_max(g, v[u].y);
            g = bf16x2_max(g, v[u].z); g = bf16x2_max(g, v[u].w);
        }
        L.pm = g;
        L.raise(fmaxf(od_bf16_lo(g), od_bf16_hi(g)), scale);
    } else {
        float gm = -INFINITY;
#pragma unroll
        for (int u = 0; u < N; ++u) {
            gm = fmaxf(gm, fmaxf(fmaxf(__uint_as_float(v[u].x), __uint_as_float(v[u].y)),
                                 fmaxf(__uint_as_float(v[u].z), __uint_as_float(v[u].w))));
        }
        L.mx = fmaxf(L.mx, gm);
        L.raise(gm, scale);
    }
    const uint64_t scale2 = f2_pack(scale, scale), nc2 = f2_pack(-L.c, -L.c);
    uint64_t a0 = 0ull, a1 = 0ull;                          // two pairs of zeros
#pragma unroll
    for (int u = 0; u < N; ++u) {
        if (DTYPE == OD_BF16) {
            a0 = f2_exp_acc(a0, od_bf16_lo(v[u].x), od_bf16_hi(v[u].x), scale2, nc2);
            a1 = f2_exp_acc(a1, od_bf16_lo(v[u].y), od_bf16_hi(v[u].y), scale2, nc2);
            a0 = f2_exp_acc(a0, od_bf16_lo(v[u].z), od_bf16_hi(v[u].z), scale2, nc2);
            a1 = f2_exp_acc(a1, od_bf16_lo(v[u].w), od_bf16_hi(v[u].w), scale2, nc2);
        } else {
            a0 = f2_exp_acc(a0, __uint_as_float(v[u].x), __uint_as_float(v[u].y), scale2, nc2);
            a1 = f2_exp_acc(a1, __uint_as_float(v[u].z), __uint_as_float(v[u].w), scale2, nc2);
        }
    }
    float s0, s1;
    f2_unpack(f2_add(a0, a1), s0, s1);
    L.s += s0 + s1;
}

template <int DTYPE>
__device__ __forceinline__ void absorb_one(Lane<DTYPE> &L, float x, float scale)
{
    if (DTYPE == OD_BF16) {
        // x is a bf16 value: keep the packed maximum exact
        L.pm = bf16x2_max(L.pm, __float_as_uint(x) >> 16 | 0xFF800000u);
    } else {
        L.mx = fmaxf(L.mx, x);
    }
    L.raise(x, scale);
    L.s += od_ex2(fmaf(x, scale, -L.c));
}

// the first n (1..U, the same for the whole warp) loads of a group
template <int TW>
__device__ __forceinline__ void load_group(uint4 (&x)[U], const uint4 *p, int n)
{
#pragma unroll
    for (int u = 0; u < U; ++u)
        if (u < n) x[u] = ld_stream(p + u * TW * 32);
}

template <int DTYPE>
__device__ __forceinline__ void absorb_group(Lane<DTYPE> &L, const uint4 (&x)[U], int n, float scale)
{
    static_assert(U == 4, "one case per group size");
    if (n == 4) absorb<DTYPE, 4>(L, x, scale);
    else if (n == 3) absorb<DTYPE, 3>(L, x, scale);
    else if (n == 2) absorb<DTYPE, 2>(L, x, scale);
    else absorb<DTYPE, 1>(L, x, scale);
}

// Units [v0, v1) of row (b, r) by the whole block; warp w stores its partial to dst[w]
// (global or shared memory).
template <int DTYPE, int TW>
__device__ __forceinline__ void block_segment(const VerifyArgs &a, int b, int r, int v0, int v1, float4 *dst)
{
    constexpr int VEC = DTYPE == OD_BF16 ? 8 : 4;          // elements per 16 bytes
    constexpr size_t ESZ = DTYPE == OD_BF16 ? 2 : 4;
    const float T = a.temperature[b];
    const float scale = (T > 0.f) ? 1.4426950408889634f / T : 0.f;   // log2(e)/T
    const char *row = (const char *)a.logits + ((size_t)b * a.seq_stride + (size_t)r * a.row_stride) * ESZ;
    Lane<DTYPE> L;
    L.reset();
    // A warp owns whole units (512 bytes, 16 per lane): units v0 + warp, + TW, ...
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int full_vecs = a.v_p / VEC;                     // whole 16-byte vectors in the row
    const int full_units = full_vecs >> 5;                 // units whose 32 lanes are all inside
    const int v1f = v1 < full_units ? v1 : full_units;
    const int v = v0 + warp;
    const uint4 *p = (const uint4 *)row + (size_t)v * 32 + lane;
    // Software pipeline over groups of U units: the loads of the next group are
    // issued before the current group is folded in, so a warp always has loads in
    // flight while it keeps the exp pipe busy (warps of a block move in lockstep,
    // they cannot hide one another's latency). The last group holds what is left
    // (1..U units) and is requested like any other, one group ahead; no lane ever
    // computes on padding. Only the row's last unit can be ragged (lanes past the
    // end of the row, or a final piece under 16 bytes).
    int cnt = v < v1f ? (v1f - v + TW - 1) / TW : 0;   // this warp's whole units
    if (cnt > 0) {
        uint4 xa[U], xb[U];
        int na = cnt < U ? cnt : U, nb = 0;
        load_group<TW>(xa, p, na);
        cnt -= na; p += U * TW * 32;
        for (;;) {
            if (cnt == 0) { absorb_group<DTYPE>(L, xa, na, scale); break; }
            nb = cnt < U ? cnt : U;
            load_group<TW>(xb, p, nb);
            cnt -= nb; p += U * TW * 32;
            absorb<DTYPE, U>(L, xa, scale);
            if (cnt == 0) { absorb_group<DTYPE>(L, xb, nb, scale); break; }
            na = cnt < U ? cnt : U;
            load_group<TW>(xa, p, na);
            cnt -= na; p += U * TW * 32;
            absorb<DTYPE, U>(L, xb, scale);
        }
    }
    if (v1 > full_units && warp == ((full_units - v0) & (TW - 1))) {
        // the row's ragged last unit (v1 == W here): whole vectors, then single elements
        const int i = full_units * 32 + lane;
        if (i < full_vecs) {
            uint4 x[1];
            x[0] = ld_stream((const uint4 *)row + i);
            absorb<DTYPE, 1>(L, x, scale);
        }
        const int e = full_vecs * VEC + lane;
        if (e < a.v_p) absorb_one<DTYPE>(L, od_load_logit<DTYPE>(row, e), scale);
    }
    // every warp publishes its own partial: no block barrier anywhere in the stream
    float c = L.c, s = L.s, mx = L.max_seen();
    warp_merge(c, s, mx);
    if (lane == 0) dst[warp] = make_float4(c, s, mx, 0.f);
}

// n / d for n < 2^31 and a divisor known at launch: with l = ceil(log2 d) and
// mul = ceil(2^(31+l) / d) < 2^32, floor(n / d) = (n * mul) >> (31 + l) exactly, because
// mul * d exceeds 2^(31+l) by less than d <= 2^l. mul == 0 stands for d == 1.
__device__ __forceinline__ uint32_t div_by(uint32_t n, uint32_t mul, uint32_t sh)
{
    return mul ? __umulhi(n, mul) >> sh : n;
}

// Row rho of space B (rows 1..m_b of every sequence, in sequence order): its sequence b,
// its row r and m_b. Lane l holds the sequences [i0, i1) and `excl`, the number of rows
// of space B before them; exactly one lane finds rho among its own (rho < rows of space
// B), and a shuffle tells the others. With at most two sequences per lane their m are in
// registers (m0, m1): no shared memory and no barrier, a warp needs nothing from the rest
// of its block; larger batches read the block's copy s_m.
__device__ __forceinline__ void find_row(const int32_t *s_m, uint32_t rho, int i0, int i1, uint32_t excl,
                                         uint32_t m0, uint32_t m1, int &b, int &r, int &mb)
{
    uint32_t run = excl;
    int hit = -1;
    if (s_m == nullptr) {
        // the lane's (clamped) m are in registers: m0, m1 (0 where the lane has no sequence)
        if (rho - run < m0) hit = i0 | (int)(1u + rho - run) << 12 | (int)m0 << 20;
        run += m0;
        if (rho - run < m1) hit = (i0 + 1) | (int)(1u + rho - run) << 12 | (int)m1 << 20;
    } else {
#pragma unroll 1
        for (int i = i0; i < i1; ++i) {
            const uint32_t mi = s_m[i];
            if (rho - run < mi) hit = i | (int)(1u + rho - run) << 12 | (int)mi << 20;   // run <= rho < run + mi
            run += mi;
        }
    }
    const unsigned found = __ballot_sync(0xFFFFFFFFu, hit >= 0);
    hit = __shfl_sync(0xFFFFFFFFu, hit, __ffs(found) - 1);
    b = hit & 0xFFF; r = hit >> 12 & 0xFF; mb = hit >> 20;
}
static_assert(OD_VERIFY_MAX_B <= 4096 && OD_MAX_K < 255 && OD_MAX_K <= 255, "find_row packs (b, r, m_b) into one word");

// Block g's span of space A (row 0 of every sequence, W units each, span_a units per block):
// flat units [lo, hi), the first one being unit v0 of sequence b0; a row that starts in the
// span has its segment 0 here, the row the span starts inside has segment seg0 here.
__device__ __forceinline__ void span_of_space_a(const VerifyArgs &a, uint32_t g, uint32_t &lo, uint32_t &hi,
                                                uint32_t &b0, uint32_t &v0, uint32_t &seg0)
{
    const uint32_t W = (uint32_t)a.W, tot = (uint32_t)a.B * W;
    lo = g * (uint32_t)a.span_a;
    if (lo > tot) lo = tot;
    hi = lo + (uint32_t)a.span_a;
    if (hi > tot) hi = tot;
    b0 = div_by(lo, a.w_mul, a.w_sh);
    v0 = lo - b0 * W;
    seg0 = g - (lo - v0) / (uint32_t)a.span_a;
}

// first of the partial slots (one per warp of a block) of segment `seg` of row (b, r)
__device__ __forceinline__ float4 *partial_slot(const VerifyArgs &a, int b, int r, int seg)
{
    return a.partials + ((size_t)b * (a.K_max + 1) + r) * OD_VERIFY_SEG_MAX + seg * a.seg_warps;
}

// 56 registers, not 64: four resident blocks then leave an eighth of the SM's register
// file free, enough for a block of the (small) kernel before or after this one in
// the stream to be resident at the same time under programmatic dependent launch.
template <int DTYPE, int TW>
__global__ void __maxnreg__(OD_VERIFY_MAXNREG)
od_verify_stream_kernel(const VerifyArgs a)
{
    constexpr int THREADS = TW * 32;
    __shared__ float4 s_park[A_PARK][TW];
    __shared__ int32_t s_m[OD_VERIFY_MAX_B];               // clamped m_b, batches of more than 64 sequences only

    // Flat unit indices stay below 2^31 (the launcher checks). What a block does between
    // griddepcontrol.wait and its first load of space B is the one stretch of this kernel
    // in which the memory system has nothing to do, and with 32 warps per multiprocessor
    // that run the same code every instruction there costs eight issue cycles: the
    // walk below uses 32-bit arithmetic, multiplications in place of the divisions by W and
    // by the grid size, registers and shuffles in place of shared memory and barriers.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t g = blockIdx.x;
    const uint32_t W = (uint32_t)a.W;

    // ---- space A (row 0 of every sequence). Nothing here depends on the translation
    // kernel (logits and temperatures are inputs of the step), so where those inputs are
    // known to be complete (a_early) this phase runs, under programmatic dependent launch,
    // while the launch in front is still at work. Its partials wait in shared memory: the
    // scratch in global memory may still be read by the previous launch's decide kernel
    // until griddepcontrol.wait returns.
    uint32_t a_lo, a_hi, a_b0, a_v0, a_seg0;
    span_of_space_a(a, g, a_lo, a_hi, a_b0, a_v0, a_seg0);
    const bool early = a.a_early != 0;                      // the span has at most A_PARK segments
    if (early && a_lo < a_hi) {
        uint32_t f = a_lo, b = a_b0, v0 = a_v0;
        int k = 0;
        while (f < a_hi) {
            uint32_t n = a_hi - f;
            if (n > W - v0) n = W - v0;
            block_segment<DTYPE, TW>(a, (int)b, 0, (int)v0, (int)(v0 + n), s_park[k++]);
            f += n; ++b; v0 = 0;
        }
    }
    // lane l of every warp will hold the sequences [i0, i1)
    const int per = (a.B + 31) >> 5;
    const int i0 = lane * per < a.B ? lane * per : a.B;
    const int i1 = i0 + per < a.B ? i0 + per : a.B;
    const uint32_t chunk = (uint32_t)a.n_chunks - 1 - g;    // spans of space B are handed out from the other end of the grid

    // everything below may read what the translation kernel wrote, and may write scratch
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");

    // ---- rows of space B before each lane's sequences, and in all
    uint32_t loc = 0, m0 = 0, m1 = 0;
    int32_t raw0 = 0, raw1 = 0;
    if (per <= 2) {
        if (i0 < i1) raw0 = a.m[i0];
        if (i0 + 1 < i1) raw1 = a.m[i0 + 1];
    }
    // ---- the parked partials of space A: every warp hands over its own (its lane 0 wrote
    // them) while the loads of m are on their way: the warp has nothing else to do
    if (early && lane == 0) {
        uint32_t f = a_lo, b = a_b0, v0 = a_v0, seg = a_seg0;
        int k = 0;
        while (f < a_hi) {
            uint32_t n = a_hi - f;
            if (n > W - v0) n = W - v0;
            partial_slot(a, (int)b, 0, (int)seg)[warp] = s_park[k][warp];
            ++k; f += n; ++b; v0 = 0; seg = 0;
        }
    }
    if (per <= 2) {
        m0 = (uint32_t)clamp_m(raw0, a.K_max);
        m1 = (uint32_t)clamp_m(raw1, a.K_max);
        loc = m0 + m1;
    } else {
        // more than 64 sequences: the block reads m once into shared memory (a load that is
        // repeated goes to L2 again, and a warp looks its rows up once per sequence)
        for (int i = threadIdx.x; i < a.B; i += THREADS) s_m[i] = clamp_m(a.m[i], a.K_max);
        __syncthreads();
#pragma unroll 1
        for (int i = i0; i < i1; ++i) loc += (uint32_t)s_m[i];
    }
    uint32_t inc = loc;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, off);
        if (lane >= off) inc += t;
    }
    const uint32_t rows_b = __shfl_sync(0xFFFFFFFFu, inc, 31);
    const uint32_t excl = inc - loc;

    if (!early && a_lo < a_hi) {
        uint32_t f = a_lo, b = a_b0, v0 = a_v0, seg = a_seg0;
        while (f < a_hi) {
            uint32_t n = a_hi - f;
            if (n > W - v0) n = W - v0;
            block_segment<DTYPE, TW>(a, (int)b, 0, (int)v0, (int)(v0 + n), partial_slot(a, (int)b, 0, (int)seg));
            f += n; ++b; v0 = 0; seg = 0;
        }
    }

    // ---- space B (rows 1..m_b)
    const uint32_t b_tot = rows_b * W;
    uint32_t span = div_by(b_tot + (uint32_t)a.n_chunks - 1, a.c_mul, a.c_sh);
    if (span < (uint32_t)a.span_min) span = (uint32_t)a.span_min;
    uint32_t f = chunk * span;
    if (f < b_tot) {
        uint32_t f_hi = f + span;
        if (f_hi > b_tot) f_hi = b_tot;
        uint32_t rho = div_by(f, a.w_mul, a.w_sh), v0 = f - rho * W;
        uint32_t seg = chunk - (f - v0) / span;
        int b, r, mb;
        find_row(per <= 2 ? nullptr : s_m, rho, i0, i1, excl, m0, m1, b, r, mb);
        for (;;) {
            uint32_t n = f_hi - f;
            if (n > W - v0) n = W - v0;
            block_segment<DTYPE, TW>(a, b, r, (int)v0, (int)(v0 + n), partial_slot(a, b, r, (int)seg));
            f += n;
            if (f >= f_hi) break;
            ++rho; v0 = 0; seg = 0;
            if (r < mb) ++r; else find_row(per <= 2 ? nullptr : s_m, rho, i0, i1, excl, m0, m1, b, r, mb);
        }
    }
}

// Row r of sequence b from its merged statistics (c, s, mx): row maximum and sum,
// p(t_i), the ratio and the accept / boundary bits (one thread per row).
__device__ __forceinline__ void decide_row(const VerifyArgs &a, int b, int r, int mb, float c, float s, float mx,
                                           float scale, bool t_ok, float x_t, float q, float u,
                                           unsigned int *s_bits)
{
    const int row_slot = b * (a.K_max + 1) + r;
    const float M = mx;
    const float S = row_sum_of(c, s, mx, scale);        // sum of exp2((x - M)*scale)
    a.row_max[row_slot] = M;
    a.row_sum[row_slot] = S;
    if (!(S > 0.f) || !(S <= FLT_MAX)) atomicOr(&s_bits[1], 1u);   // not finite and positive
    if (r < mb) {
        const size_t o = (size_t)b * a.K_max + r;
        const Acceptance d = accept_position(M, S, scale, t_ok, x_t, q, u);
        a.p_sel[o] = d.p;
        a.ratio[o] = d.ratio;
        unsigned int bits = 0;
        if (d.accept) bits |= 1u << r;
        if (d.boundary) bits |= 1u << (16 + r);
        if (bits) atomicOr(&s_bits[0], bits);
    }
}

// The accepted prefix of sequence b from the rows' bits, by warp 0: lane k holds
// span_len[b, k] (loaded before the kernel waited), so nothing is loaded here.
__device__ __forceinline__ void decide_prefix(const VerifyArgs &a, int b, int mb, bool bad_T,
                                              const unsigned int *s_bits, int lane, int32_t my_span)
{
    const unsigned int all = s_bits[0];
    int n = 0;
    while (n < mb && (all >> n & 1u)) ++n;
    int nd = lane < n ? my_span : 0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) nd += __shfl_xor_sync(0xFFFFFFFFu, nd, off);
    if (lane != 0) return;
    uint32_t f = (all >> 16) & OD_VF_BOUNDARY_MASK;
    if (s_bits[1] & 1u) f |= OD_VF_NONFINITE;
    if (bad_T) { f |= OD_VF_BAD_TEMPERATURE; n = 0; nd = 0; }
    a.n_accepted[b] = n;
    a.n_draft_accepted[b] = nd;
    a.flags[b] = f;
}

// One block per sequence, warp r = row r (blockDim = 32 * (K_max + 1)).
// SHARD: the rows are the columns [col0, col0 + v_p) of the full rows; the merged
// statistics of a row are stored as this shard's record and nothing is decided.
template <int DTYPE, bool SHARD>
__global__ void __launch_bounds__(32 * (OD_MAX_K + 1))
od_verify_decide_kernel(const VerifyArgs a)
{
    constexpr size_t ESZ = DTYPE == OD_BF16 ? 2 : 4;
    __shared__ int32_t s_part[2][OD_MAX_K + 1];
    __shared__ unsigned int s_bits[2];

    // The next kernel of the stream may be placed as soon as this grid is resident: what
    // it does before its own griddepcontrol.wait (the sampler: nothing; the next step's
    // stream kernel: row 0 of its sequences) then fills the multiprocessors that the
    // stream kernel's last blocks leave idle. Its wait still covers this whole grid.
    asm volatile("griddepcontrol.launch_dependents;");

    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, r = threadIdx.x >> 5;
    const uint32_t W = (uint32_t)a.W;

    // ---- before the stream kernel has finished: everything that does not depend on it.
    // (m, the target ids and q' come from the translation kernel, which was complete
    // before any block of the stream kernel let this grid start.)
    int before = 0, total = 0;                               // sums of clamped m over [0, b) and [0, B)
    for (int i = threadIdx.x; i < a.B; i += blockDim.x) {
        const int v = clamp_m(a.m[i], a.K_max);
        total += v;
        if (i < b) before += v;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        before += __shfl_xor_sync(0xFFFFFFFFu, before, off);
        total += __shfl_xor_sync(0xFFFFFFFFu, total, off);
    }
    if (lane == 0) { s_part[0][r] = before; s_part[1][r] = total; }
    if (threadIdx.x == 0) { s_bits[0] = 0; s_bits[1] = 0; }
    const int mb = clamp_m(a.m[b], a.K_max);
    const float T = a.temperature[b];
    const bool bad_T = !(T > 0.f);
    const float scale = bad_T ? 0.f : 1.4426950408889634f / T;
    const char *row = (const char *)a.logits + ((size_t)b * a.seq_stride + (size_t)r * a.row_stride) * ESZ;
    float x_t = 0.f, q = 0.f, u = 0.f;
    bool t_ok = false;
    int32_t my_span = 0;                                     // warp 0, lane k: span_len[b, k]
    if (!SHARD && r == 0 && lane < mb) my_span = a.span_len[(size_t)b * a.K_max + lane];
    if (lane == 0 && r < mb) {
        const size_t o = (size_t)b * a.K_max + r;
        const int32_t t = a.tgt_ids[o] - (SHARD ? a.col0 : 0);
        t_ok = t >= 0 && t < a.v_p;
        if (t_ok) x_t = od_load_logit<DTYPE>(row, t);
        if (!SHARD) {
            q = a.q_prime[o];
            u = od_uniform(a.seed[b], a.step, (uint32_t)r, 0u);
        }
    }
    __syncthreads();
    before = 0; total = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { before += s_part[0][w]; total += s_part[1][w]; }

    int nseg = 0;
    if (r <= mb) {
        if (r == 0) nseg = row_segments((uint32_t)b, W, (uint32_t)a.span_a);
        else nseg = row_segments((uint32_t)(before + r - 1), W,
                                 span_of_space_b((uint32_t)total, W, (uint32_t)a.n_chunks, (uint32_t)a.span_min));
    }

    // ---- the partials
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (r <= mb) {
        const int row_slot = b * (a.K_max + 1) + r;
        StreamPlan plan;
        plan.partials = a.partials;
        plan.seg_warps = a.seg_warps;
        float c, s, mx;
        merge_row_partials(plan, row_slot, nseg, lane, c, s, mx);
        if (SHARD) {
            if (lane == 0) a.stats[row_slot] = make_float4(c, s, mx, t_ok ? x_t : -INFINITY);
        } else {
            if (lane == 0) decide_row(a, b, r, mb, c, s, mx, scale, t_ok, x_t, q, u, s_bits);
        }
    }
    if (SHARD) return;
    __syncthreads();
    if (r == 0) decide_prefix(a, b, mb, bad_T, s_bits, lane, my_span);
}

// Vocabulary shards, after the exchange: one block per sequence, warp r = row r merges
// the row's records of all shards (in shard order) and decides as above. x[t_i] is the
// one finite entry among the records (the shard that owns t_i), or -inf.
__global__ void __launch_bounds__(32 * (OD_MAX_K + 1))
od_verify_finish_kernel(const VerifyArgs a)
{
    __shared__ unsigned int s_bits[2];
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, r = threadIdx.x >> 5;
    if (threadIdx.x == 0) { s_bits[0] = 0; s_bits[1] = 0; }
    const int mb = clamp_m(a.m[b], a.K_max);
    const float T = a.temperature[b];
    const bool bad_T = !(T > 0.f);
    const float scale = bad_T ? 0.f : 1.4426950408889634f / T;
    float q = 0.f, u = 0.f;
    bool t_ok = false;
    int32_t my_span = 0;
    if (r == 0 && lane < mb) my_span = a.span_len[(size_t)b * a.K_max + lane];
    if (lane == 0 && r < mb) {
        const size_t o = (size_t)b * a.K_max + r;
        const int32_t t = a.tgt_ids[o];
        t_ok = t >= 0 && t < a.v_p;
        q = a.q_prime[o];
        u = od_uniform(a.seed[b], a.step, (uint32_t)r, 0u);
    }
    __syncthreads();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    if (r <= mb) {
        const int row_slot = b * (a.K_max + 1) + r;
        float c = -FLT_MAX, s = 0.f, mx = -INFINITY, x_t = -INFINITY;
        for (int k = lane; k < a.n_shards; k += 32) {
            const float4 p = __ldcg(a.stats_all + (size_t)k * a.stats_rows + row_slot);
            pair_merge(c, s, p.x, p.y);
            mx = fmaxf(mx, p.z);
            x_t = fmaxf(x_t, p.w);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) x_t = fmaxf(x_t, __shfl_xor_sync(0xFFFFFFFFu, x_t, off));
        warp_merge(c, s, mx);
        if (lane == 0) decide_row(a, b, r, mb, c, s, mx, scale, t_ok, x_t, q, u, s_bits);
    }
    __syncthreads();
    if (r == 0) decide_prefix(a, b, mb, bad_T, s_bits, lane, my_span);
}

template <typename Kern>
cudaError_t launch(Kern kern, unsigned grid, unsigned block, cudaStream_t s, bool pdl, const VerifyArgs &a)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

}  // namespace

// multiplier and shift of div_by for the divisor d >= 1
static void fast_div(uint32_t d, uint32_t &mul, uint32_t &sh)
{
    if (d <= 1) { mul = 0; sh = 0; return; }
    uint32_t l = 0;
    while (((uint64_t)1 << l) < d) ++l;                     // l = ceil(log2 d) >= 1
    const unsigned __int128 num = (unsigned __int128)1 << (31 + l);
    mul = (uint32_t)((num + d - 1) / d);
    sh = l - 1;
}

// the stream kernel in the block shape the plan chose
template <int DTYPE>
static cudaError_t launch_stream(const VerifyArgs &a, cudaStream_t s, bool pdl)
{
    return a.seg_warps == WIDE_WARPS
        ? launch(od_verify_stream_kernel<DTYPE, WIDE_WARPS>, (unsigned)a.n_chunks, WIDE_WARPS * 32, s, pdl, a)
        : launch(od_verify_stream_kernel<DTYPE, NARROW_WARPS>, (unsigned)a.n_chunks, NARROW_WARPS * 32, s, pdl, a);
}

// Launch plan of the stream kernel for `nb` sequences whose rows hold `v_len` elements.
static void plan_stream(const od_ctx *c, int32_t nb, int32_t K_max, int32_t v_len, int32_t dtype, bool early,
                        VerifyArgs &a)
{
    const int64_t esz = dtype == OD_BF16 ? 2 : 4;
    const int64_t row_bytes = (int64_t)v_len * esz;
    const int32_t W = (int32_t)((row_bytes + 511) / 512);
    const int32_t warps = W >= WIDE_MIN_UNITS ? WIDE_WARPS : NARROW_WARPS;
    // a row is cut into at most OD_VERIFY_SEG_MAX / warps block segments (one partial per warp each)
    const int MAX_BLOCK_SEGS = OD_VERIFY_SEG_MAX / warps;
    const int32_t span_min = (W + MAX_BLOCK_SEGS - 2) / (MAX_BLOCK_SEGS - 1);
    // one resident wave, and no more blocks than the most this slice can need
    const int64_t max_units = (int64_t)nb * (K_max + 1) * W;
    // one resident wave: 32 warps per multiprocessor at 56 registers
    int64_t grid = c->opt_verify_grid > 0 ? c->opt_verify_grid
                                          : (int64_t)c->sm_count * OD_VERIFY_BLOCKS_PER_SM * NARROW_WARPS / warps;
    const int64_t need = max_units / span_min + 1;
    if (grid > need) grid = need;
    if (grid < 1) grid = 1;
    a.B = nb; a.K_max = K_max; a.v_p = v_len;
    a.W = W; a.n_chunks = (int32_t)grid; a.span_min = span_min; a.seg_warps = warps;
    int64_t span_a = ((int64_t)nb * W + grid - 1) / grid;
    if (span_a < span_min) span_a = span_min;
    a.span_a = (int32_t)span_a;
    a.a_early = early && span_a / W + 2 <= A_PARK;
    fast_div((uint32_t)W, a.w_mul, a.w_sh);
    fast_div((uint32_t)grid, a.c_mul, a.c_sh);
}

// batches beyond the shared-memory prefix table go in slices; a slice's flat
// unit indices (plus one span of slack) must fit 32 bits
static int32_t slice_of(int32_t K_max, int32_t v_len, int32_t dtype)
{
    const int64_t W = ((int64_t)v_len * (dtype == OD_BF16 ? 2 : 4) + 511) / 512;
    int32_t slice = OD_VERIFY_MAX_B;
    while (slice > 1 && (int64_t)slice * (K_max + 1) * W > (int64_t)1 << 30) slice >>= 1;
    return slice;
}

int32_t od_verify_slice(int32_t K_max, int32_t v_len, int32_t dtype) { return slice_of(K_max, v_len, dtype); }

// The streaming pass alone, for a batch that fits one launch (B <= od_verify_slice): the
// caller's next kernel merges the partials itself (od_step).
cudaError_t od_launch_verify_stream(od_ctx *c, int32_t B, int32_t K_max, const void *logits, int32_t dtype,
                                    int64_t row_stride, int64_t seq_stride, const int32_t *m,
                                    const float *temperature, od_fused_verify *plan, cudaStream_t s)
{
    c->last_was_map = false;
    VerifyArgs a = {};
    plan_stream(c, B, K_max, c->v_p, dtype, c->verify_early, a);
    a.logits = logits; a.row_stride = row_stride; a.seq_stride = seq_stride;
    a.m = m; a.temperature = temperature;
    a.partials = c->d_partials;
    c->info[0] = a.n_chunks;
    c->info[1] = a.span_a;
    plan->W = a.W; plan->n_chunks = a.n_chunks; plan->span_min = a.span_min; plan->span_a = a.span_a;
    plan->seg_warps = a.seg_warps;
    const bool pdl = c->opt_pdl != 0;
    return dtype == OD_BF16 ? launch_stream<OD_BF16>(a, s, pdl)
                            : launch_stream<OD_F32>(a, s, pdl);
}

cudaError_t od_launch_verify(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                             int32_t dtype, int64_t row_stride, int64_t seq_stride,
                             const int32_t *tgt_ids, const float *q_prime,
                             const int32_t *span_len, const int32_t *m,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             float *row_max, float *row_sum, float *p_sel, float *ratio,
                             int32_t *n_accepted, int32_t *n_draft_accepted,
                             uint32_t *flags, cudaStream_t s)
{
    const int64_t esz = dtype == OD_BF16 ? 2 : 4;
    const int32_t slice = slice_of(K_max, c->v_p, dtype);
    c->last_was_map = false;
    for (int32_t b0 = 0; b0 < B; b0 += slice) {
        const int32_t nb = B - b0 < slice ? B - b0 : slice;
        VerifyArgs a = {};
        plan_stream(c, nb, K_max, c->v_p, dtype, c->verify_early, a);
        a.logits = (const char *)logits + (size_t)b0 * seq_stride * esz;
        a.row_stride = row_stride; a.seq_stride = seq_stride;
        a.tgt_ids = tgt_ids + (size_t)b0 * K_max; a.q_prime = q_prime + (size_t)b0 * K_max;
        a.span_len = span_len + (size_t)b0 * K_max; a.m = m + b0;
        a.temperature = temperature + b0; a.seed = seed + b0; a.step = step;
        a.row_max = row_max + (size_t)b0 * (K_max + 1); a.row_sum = row_sum + (size_t)b0 * (K_max + 1);
        a.p_sel = p_sel + (size_t)b0 * K_max; a.ratio = ratio + (size_t)b0 * K_max;
        a.n_accepted = n_accepted + b0; a.n_draft_accepted = n_draft_accepted + b0;
        a.flags = flags + b0;
        a.partials = c->d_partials;
        c->info[0] = a.n_chunks;
        c->info[1] = a.span_a;

        const bool pdl = c->opt_pdl != 0;
        cudaError_t e = dtype == OD_BF16
            ? launch_stream<OD_BF16>(a, s, pdl)
            : launch_stream<OD_F32>(a, s, pdl);
        if (e != cudaSuccess) return e;
        const unsigned dthreads = 32u * (unsigned)(K_max + 1);
        e = dtype == OD_BF16
            ? launch(od_verify_decide_kernel<OD_BF16, false>, (unsigned)nb, dthreads, s, pdl, a)
            : launch(od_verify_decide_kernel<OD_F32, false>, (unsigned)nb, dthreads, s, pdl, a);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// One vocabulary shard: the statistics of columns [shard_lo, shard_lo + shard_len) of
// every row, one record per row into stats[B * (K_max + 1)].
cudaError_t od_launch_verify_shard_stats(od_ctx *c, int32_t B, int32_t K_max, int32_t shard_lo,
                                         int32_t shard_len, const void *logits, int32_t dtype,
                                         int64_t row_stride, int64_t seq_stride, const int32_t *tgt_ids,
                                         const int32_t *m, const float *temperature, float *stats,
                                         cudaStream_t s)
{
    const int64_t esz = dtype == OD_BF16 ? 2 : 4;
    const int32_t slice = slice_of(K_max, shard_len, dtype);
    c->last_was_map = false;
    for (int32_t b0 = 0; b0 < B; b0 += slice) {
        const int32_t nb = B - b0 < slice ? B - b0 : slice;
        VerifyArgs a = {};
        plan_stream(c, nb, K_max, shard_len, dtype, c->verify_early, a);
        a.logits = (const char *)logits + (size_t)b0 * seq_stride * esz;
        a.row_stride = row_stride; a.seq_stride = seq_stride;
        a.tgt_ids = tgt_ids + (size_t)b0 * K_max; a.m = m + b0;
        a.temperature = temperature + b0;
        a.partials = c->d_partials;
        a.col0 = shard_lo;
        a.stats = (float4 *)stats + (size_t)b0 * (K_max + 1);
        c->info[0] = a.n_chunks;
        c->info[1] = a.span_a;
        const bool pdl = c->opt_pdl != 0;
        cudaError_t e = dtype == OD_BF16
            ? launch_stream<OD_BF16>(a, s, pdl)
            : launch_stream<OD_F32>(a, s, pdl);
        if (e != cudaSuccess) return e;
        const unsigned dthreads = 32u * (unsigned)(K_max + 1);
        e = dtype == OD_BF16
            ? launch(od_verify_decide_kernel<OD_BF16, true>, (unsigned)nb, dthreads, s, pdl, a)
            : launch(od_verify_decide_kernel<OD_F32, true>, (unsigned)nb, dthreads, s, pdl, a);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// After the exchange: merge the records of all shards and decide.
cudaError_t od_launch_verify_shard_finish(od_ctx *c, int32_t B, int32_t K_max, int32_t n_shards,
                                          const float *stats_all, const int32_t *tgt_ids,
                                          const float *q_prime, const int32_t *span_len, const int32_t *m,
                                          const float *temperature, const uint64_t *seed, uint64_t step,
                                          float *row_max, float *row_sum, float *p_sel, float *ratio,
                                          int32_t *n_accepted, int32_t *n_draft_accepted, uint32_t *flags,
                                          cudaStream_t s)
{
    c->last_was_map = false;
    if (B == 0) return cudaSuccess;
    VerifyArgs a = {};
    a.B = B; a.K_max = K_max; a.v_p = c->v_p;
    a.tgt_ids = tgt_ids; a.q_prime = q_prime; a.span_len = span_len; a.m = m;
    a.temperature = temperature; a.seed = seed; a.step = step;
    a.row_max = row_max; a.row_sum = row_sum; a.p_sel = p_sel; a.ratio = ratio;
    a.n_accepted = n_accepted; a.n_draft_accepted = n_draft_accepted; a.flags = flags;
    a.n_shards = n_shards;
    a.stats_all = (const float4 *)stats_all;
    a.stats_rows = (int64_t)B * (K_max + 1);
    return launch(od_verify_finish_kernel, (unsigned)B, 32u * (unsigned)(K_max + 1), s, c->opt_pdl != 0, a);
}
