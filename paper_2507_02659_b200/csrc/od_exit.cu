// Adaptive-drafting exit rule (Section 3.3, Eq. (4)-(6)): from the acceptance head's
// outputs f_phi(e_i) of the proposed tokens, the probability that some token up to
// k is rejected, 1 - prod_{i<=k} sigmoid(f_i), and the draft length: the first k at
// which that probability exceeds gamma (all available tokens if it never does).
// The result is the ragged draft_len that od_map_proposals takes.
//
// A few dozen flops per sequence: one thread per sequence, fp32, the product taken
// in token order exactly as the definition reads.
#include "od_common.cuh"

namespace {

__device__ __forceinline__ float sigmoid_f32(float x)
{
    // the two branches avoid overflow of exp for large |x|
    if (x >= 0.f) return 1.f / (1.f + expf(-x));
    const float e = expf(x);
    return e / (1.f + e);
}

__global__ void od_exit_kernel(int32_t B, int32_t K_max, const float *__restrict__ head_logits,
                               const int32_t *__restrict__ avail_len, float gamma,
                               int32_t *__restrict__ draft_len, float *__restrict__ reject_prob,
                               uint32_t *__restrict__ flags)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int n = avail_len ? avail_len[b] : K_max;
    n = n < 0 ? 0 : (n > K_max ? K_max : n);
    float keep = 1.f;                                      // running product of Eq. (5)
    int length = n;
    bool fired = false;
    uint32_t f = 0;
    for (int i = 0; i < K_max; ++i) {
        float rej = 0.f;
        if (i < n) {
            keep *= sigmoid_f32(head_logits[(size_t)b * K_max + i]);
            rej = 1.f - keep;
            if (!fired) {
                if (fabsf(rej - gamma) <= OD_TAU_EXIT) f |= 1u << i;   // fp32 may land on the other side
                if (rej > gamma) { length = i + 1; fired = true; }
            }
        }
        if (reject_prob) reject_prob[(size_t)b * K_max + i] = rej;
    }
    draft_len[b] = length;
    if (flags) flags[b] = f;
}

}  // namespace

cudaError_t od_launch_exit(int32_t B, int32_t K_max, const float *head_logits, const int32_t *avail_len,
                           float gamma, int32_t *draft_len, float *reject_prob, uint32_t *flags,
                           cudaStream_t s)
{
    if (B == 0) return cudaSuccess;
    const int threads = 128;
    od_exit_kernel<<<(B + threads - 1) / threads, threads, 0, s>>>(B, K_max, head_logits, avail_len, gamma,
                                                                   draft_len, reject_prob, flags);
    return cudaGetLastError();
}
