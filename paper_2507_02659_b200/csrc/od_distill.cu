// Hybrid cross-vocabulary distillation loss (Section 3.2, Eq. (3)) and its gradient
// with respect to the drafter's logits, per proposed draft position:
//   directly mapped token (its piece of the translated proposal has one sub-token,
//   target position i):   L = KL(q' || p_i) = sum over mapped draft ids d of
//                             q(d) * (ln q(d) - ln p_i(map[d]))
//   sub-token of a cached n-gram:   L = -lambda * ln q(d_j)   (lambda constant, or the
//                             verified target probability of the n-gram)
//   not translated:       L = 0.
// With q = softmax(z):  KL:  dL/dz(d) = q(d) * (g(d) - sum_e q(e) g(e)),
//                            g(d) = [d mapped] * (ln q(d) - ln p(map[d]) + 1)
//                       NLL: dL/dz(d) = lambda * (q(d) - [d == d_j]).
// ln p_i(t) = (x_t - M_i)/T - ln S_i reuses the row statistics od_verify produced, so
// the target row is only gathered at the mapped ids, never streamed again.
//
// One block of 512 threads per (sequence, draft position), two resident per SM so
// that a whole batch is one wave; two sweeps over the draft vocabulary: sums, with
// q(d) g(d) parked in the gradient row, then the gradient (which re-reads q and the
// parked values from cache). Reads are coalesced except the one gathered logit per
// mapped id, which touches practically every sector of the target row. Bound by HBM:
// the drafter's row and the target row in, the gradient row out.
#include <float.h>

#include "od_common.cuh"

namespace {

constexpr int THREADS = 512;

struct DistillArgs {
    int32_t B, K_max, v_q, v_p;
    const float *q_rows;
    const int32_t *draft_ids, *tgt_ids, *span_start, *span_len, *m;
    const void *logits;
    int64_t row_stride, seq_stride;
    const float *row_max, *row_sum, *p_sel, *temperature;
    const int32_t *vocab_map;
    float lambda;
    int32_t lambda_mode;
    float *loss, *grad;
};

// log2 on the special-function unit (relative error about 2^-22; the terms it enters are
// weighted by q, so the loss and the gradient see it far below their fp32 rounding)
__device__ __forceinline__ float lg2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ double block_sum(double v, double *s_red)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < THREADS / 32; ++w) t += s_red[w];   // the same order in every thread
    return t;
}

// VEC4: the draft vocabulary is a multiple of 4 and the rows are 16-byte aligned, so the
// coalesced accesses (map, q, gradient) move four ids per instruction.
template <int DTYPE, bool VEC4>
__global__ void __launch_bounds__(THREADS, 2)
od_distill_kernel(const DistillArgs a)
{
    __shared__ double s_red[THREADS / 32];
    const int b = blockIdx.y, j = blockIdx.x;
    const int K = a.K_max;
    int mb = a.m[b];
    mb = mb < 0 ? 0 : (mb > K ? K : mb);
    // the piece of the translated proposal that covers draft position j, if any
    // (thread i looks at piece i, so the loads go out together)
    __shared__ int s_piece, s_plen;
    if (threadIdx.x == 0) { s_piece = -1; s_plen = 0; }
    __syncthreads();
    if ((int)threadIdx.x < mb) {
        const int s0 = a.span_start[(size_t)b * K + threadIdx.x], L = a.span_len[(size_t)b * K + threadIdx.x];
        if (j >= s0 && j < s0 + L) { s_piece = (int)threadIdx.x; s_plen = L; }
    }
    __syncthreads();
    const int piece = s_piece, plen = s_plen;
    const float *q = a.q_rows + ((size_t)b * K + j) * a.v_q;
    float *grad = a.grad ? a.grad + ((size_t)b * K + j) * a.v_q : nullptr;
    const float T = a.temperature[b];
    if (piece < 0 || !(T > 0.f)) {                           // not translated: no loss, no gradient
        if (threadIdx.x == 0) a.loss[(size_t)b * K + j] = 0.f;
        if (grad)
            for (int d = threadIdx.x; d < a.v_q; d += THREADS) grad[d] = 0.f;
        return;
    }
    if (plen >= 2) {
        // ---- a sub-token of a cached n-gram: -w ln q(d_j)
        const int32_t dj = a.draft_ids[(size_t)b * K + j];
        const float w = a.lambda_mode == 0 ? a.lambda : a.p_sel[(size_t)b * K + piece];
        if (threadIdx.x == 0) a.loss[(size_t)b * K + j] = (dj >= 0 && dj < a.v_q) ? -w * logf(q[dj]) : 0.f;
        if (grad)
            for (int d = threadIdx.x; d < a.v_q; d += THREADS) grad[d] = w * (__ldg(q + d) - (d == dj ? 1.f : 0.f));
        return;
    }
    // ---- a directly mapped token: KL(q' || p_i) over the mapped ids
    const size_t esz = DTYPE == OD_BF16 ? 2 : 4;
    const char *row = (const char *)a.logits + ((size_t)b * a.seq_stride + (size_t)piece * a.row_stride) * esz;
    // The gathers below touch practically every 32-byte sector of the target row in no
    // particular order: have the copy engine bring the row into L2 as one sequential
    // transfer first (a no-op when od_verify has just streamed it).
    if (threadIdx.x == 0) {
        const uint32_t bytes = (uint32_t)((size_t)a.v_p * esz / 16 * 16);
        if (bytes) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(row), "r"(bytes) : "memory");
    }
    // in base 2: ln q - ln p(t) = ln 2 * (lg2 q - ((x_t - M) * log2(e)/T - lg2 S))
    const float M = a.row_max[b * (K + 1) + piece];
    const float lg2_S = lg2_approx(a.row_sum[b * (K + 1) + piece]);
    const float scale = 1.4426950408889634f / T;
    constexpr float LN2 = 0.6931471805599453f;
    // Sweep 1: g(d) = [d mapped, q(d) > 0] (ln q(d) - ln p(map[d]) + 1), the loss and
    // sum_d q(d) g(d). The loads of EB ids are issued together (map and q, then the
    // gathered logits). q(d) g(d) is parked in the gradient row itself (it stays in L2),
    // so that sweep 2 neither gathers nor takes a logarithm again.
    const bool park = grad != nullptr;
    float loss_t = 0.f, qg_t = 0.f;
    // one id: q (negative = no map), its gathered logit -> the terms of the loss and of sum q g;
    // returns q(d) g(d)
    auto term = [&](float qs, float x) -> float {
        const bool ok = qs >= FLT_MIN;                       // mapped and with (normal) mass
        const float qa = fabsf(qs);
        const float f = ok ? LN2 * (lg2_approx(qa) - fmaf(x - M, scale, -lg2_S)) : 0.f;
        const float g = ok ? f + 1.f : 0.f;
        loss_t += qa * f;
        qg_t += qa * g;
        return qa * g;
    };
    if (VEC4) {
        constexpr int EV = 4;                                // vectors of 4 ids in flight per thread
        for (int base = threadIdx.x * 4; base < a.v_q; base += THREADS * 4 * EV) {
            int4 t[EV];
            float4 qv[EV];
#pragma unroll
            for (int e = 0; e < EV; ++e) {
                const int d = base + e * THREADS * 4;
                t[e] = d < a.v_q ? __ldg((const int4 *)(a.vocab_map + d)) : make_int4(-1, -1, -1, -1);
                qv[e] = d < a.v_q ? __ldg((const float4 *)(q + d)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float x[EV][4];
#pragma unroll
            for (int e = 0; e < EV; ++e) {
                x[e][0] = od_load_logit<DTYPE>(row, t[e].x >= 0 ? t[e].x : 0);
                x[e][1] = od_load_logit<DTYPE>(row, t[e].y >= 0 ? t[e].y : 0);
                x[e][2] = od_load_logit<DTYPE>(row, t[e].z >= 0 ? t[e].z : 0);
                x[e][3] = od_load_logit<DTYPE>(row, t[e].w >= 0 ? t[e].w : 0);
            }
#pragma unroll
            for (int e = 0; e < EV; ++e) {
                const int d = base + e * THREADS * 4;
                float4 o;
                o.x = term(t[e].x < 0 ? -qv[e].x : qv[e].x, x[e][0]);
                o.y = term(t[e].y < 0 ? -qv[e].y : qv[e].y, x[e][1]);
                o.z = term(t[e].z < 0 ? -qv[e].z : qv[e].z, x[e][2]);
                o.w = term(t[e].w < 0 ? -qv[e].w : qv[e].w, x[e][3]);
                if (park && d < a.v_q) *(float4 *)(grad + d) = o;
            }
        }
    } else {
        constexpr int EB = 16;
        for (int base = threadIdx.x; base < a.v_q; base += THREADS * EB) {
            float qd[EB], x[EB];
            {
                int32_t t[EB];
#pragma unroll
                for (int e = 0; e < EB; ++e) {
                    const int d = base + e * THREADS;
                    t[e] = d < a.v_q ? __ldg(a.vocab_map + d) : -1;
                    qd[e] = d < a.v_q ? __ldg(q + d) : 0.f;
                }
#pragma unroll
                for (int e = 0; e < EB; ++e)                 // an id without a map: q = 0 drops its term below
                    if (t[e] < 0) qd[e] = -qd[e];
#pragma unroll
                for (int e = 0; e < EB; ++e) x[e] = od_load_logit<DTYPE>(row, t[e] >= 0 ? t[e] : 0);
            }
#pragma unroll
            for (int e = 0; e < EB; ++e) {
                const int d = base + e * THREADS;
                const float v = term(qd[e], x[e]);
                if (park && d < a.v_q) grad[d] = v;
            }
        }
    }
    const double loss = block_sum((double)loss_t, s_red);
    const double qg = block_sum((double)qg_t, s_red);
    if (threadIdx.x == 0) a.loss[(size_t)b * K + j] = (float)loss;
    if (grad) {
        // Sweep 2: grad(d) = q(d) g(d) - q(d) * sum_e q(e) g(e); every thread revisits the
        // ids it wrote itself, so no barrier is needed for the parked values
        const float gbar = (float)qg;
        if (VEC4) {
#pragma unroll 4
            for (int d = threadIdx.x * 4; d < a.v_q; d += THREADS * 4) {
                const float4 qq = __ldg((const float4 *)(q + d));
                float4 gv = *(float4 *)(grad + d);
                gv.x = fmaf(-qq.x, gbar, gv.x); gv.y = fmaf(-qq.y, gbar, gv.y);
                gv.z = fmaf(-qq.z, gbar, gv.z); gv.w = fmaf(-qq.w, gbar, gv.w);
                *(float4 *)(grad + d) = gv;
            }
        } else {
#pragma unroll 4
            for (int d = threadIdx.x; d < a.v_q; d += THREADS) grad[d] = fmaf(-__ldg(q + d), gbar, grad[d]);
        }
    }
}

}  // namespace

cudaError_t od_launch_distill(od_ctx *c, int32_t B, int32_t K_max, const float *q_rows,
                              const int32_t *draft_ids, const int32_t *tgt_ids, const int32_t *span_start,
                              const int32_t *span_len, const int32_t *m, const void *logits, int32_t dtype,
                              int64_t row_stride, int64_t seq_stride, const float *row_max,
                              const float *row_sum, const float *p_sel, const float *temperature,
                              float lambda, int32_t lambda_mode, float *loss, float *grad, cudaStream_t s)
{
    if (B == 0) return cudaSuccess;
    DistillArgs a;
    a.B = B; a.K_max = K_max; a.v_q = c->v_q; a.v_p = c->v_p;
    a.q_rows = q_rows; a.draft_ids = draft_ids; a.tgt_ids = tgt_ids; a.span_start = span_start;
    a.span_len = span_len; a.m = m; a.logits = logits; a.row_stride = row_stride; a.seq_stride = seq_stride;
    a.row_max = row_max; a.row_sum = row_sum; a.p_sel = p_sel; a.temperature = temperature;
    a.vocab_map = c->d_vocab_map; a.lambda = lambda; a.lambda_mode = lambda_mode; a.loss = loss; a.grad = grad;
    dim3 grid((unsigned)K_max, (unsigned)B);
    const bool vec4 = c->v_q % 4 == 0 && ((uintptr_t)q_rows & 15u) == 0 && (!grad || ((uintptr_t)grad & 15u) == 0);
    if (dtype == OD_BF16) {
        if (vec4) od_distill_kernel<OD_BF16, true><<<grid, THREADS, 0, s>>>(a);
        else od_distill_kernel<OD_BF16, false><<<grid, THREADS, 0, s>>>(a);
    } else {
        if (vec4) od_distill_kernel<OD_F32, true><<<grid, THREADS, 0, s>>>(a);
        else od_distill_kernel<OD_F32, false><<<grid, THREADS, 0, s>>>(a);
    }
    return cudaGetLastError();
}
