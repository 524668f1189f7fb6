// od_verify_noalloc: step 2 of the verification path for callers that may not
// allocate device memory (see include/omnidraft.h). It runs the same two kernels
// as od_verify; the only difference is where their scratch (the per-segment
// partials of the streaming pass) lives: in the fixed array below, which every
// GPU that loads this library holds from load time until the process exits,
// instead of in memory that od_create obtains with cudaMalloc.
#include <mutex>

#include "od_common.cuh"

namespace {

// The scratch itself: OD_NOALLOC_MAX_ROWS logit rows x OD_VERIFY_SEG_MAX partials
// of 16 bytes = 1 MiB. In host code this name is only a handle for the runtime;
// the address the kernels use comes from cudaGetSymbolAddress below.
static __device__ __align__(256) float4 g_noalloc_partials[(size_t)OD_NOALLOC_MAX_ROWS * OD_VERIFY_SEG_MAX];

constexpr int MAX_DEVICES = 64;

struct DeviceSetup {
    bool done;
    float4 *partials;       // device address of g_noalloc_partials on this device
    int sm_count;
};

std::mutex g_mutex;
DeviceSetup g_setup[MAX_DEVICES];

// First use on `device` (which must be the current device): look up the device
// address of the array and the SM count. Neither call allocates.
int32_t setup_current_device(int device, DeviceSetup *out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceSetup &d = g_setup[device];
    if (!d.done) {
        float4 *ptr = nullptr;
        if (cudaGetSymbolAddress((void **)&ptr, g_noalloc_partials) != cudaSuccess || !ptr) return OD_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1)
            return OD_ERR_CUDA;
        d.partials = ptr;
        d.sm_count = sms;
        d.done = true;
    }
    *out = d;
    return OD_OK;
}

}  // namespace

extern "C" int32_t od_verify_noalloc(int32_t target_vocab, int32_t B, int32_t K_max, const void *logits,
                                     int32_t logit_dtype, int64_t row_stride, int64_t seq_stride,
                                     const int32_t *tgt_ids, const float *q_prime,
                                     const int32_t *span_len, const int32_t *m,
                                     const float *temperature, const uint64_t *seed, uint64_t step,
                                     float *row_max, float *row_sum, float *p_sel, float *ratio,
                                     int32_t *n_accepted, int32_t *n_draft_accepted,
                                     uint32_t *verify_flags, void *stream)
{
    if (target_vocab < 1 || B < 0 || K_max < 1 || K_max > OD_MAX_K) return OD_ERR_INVALID_ARG;
    if (!logits || !tgt_ids || !q_prime || !span_len || !m || !temperature || !seed || !row_max ||
        !row_sum || !p_sel || !ratio || !n_accepted || !n_draft_accepted || !verify_flags)
        return OD_ERR_INVALID_ARG;
    if (logit_dtype != OD_F32 && logit_dtype != OD_BF16) return OD_ERR_UNSUPPORTED;
    const int64_t esz = logit_dtype == OD_BF16 ? 2 : 4;
    if (row_stride < target_vocab || seq_stride < row_stride * (K_max + 1)) return OD_ERR_INVALID_ARG;
    if (((uintptr_t)logits & 15u) != 0 || (row_stride * esz) % 16 != 0 || (seq_stride * esz) % 16 != 0)
        return OD_ERR_ALIGNMENT;
    // the fixed scratch bounds the problem size
    if (B > OD_VERIFY_MAX_B || (int64_t)B * (K_max + 1) > OD_NOALLOC_MAX_ROWS) return OD_ERR_SCRATCH_LIMIT;
    if (B == 0) return OD_OK;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return OD_ERR_CUDA;
    if (device < 0 || device >= MAX_DEVICES) return OD_ERR_UNSUPPORTED;
    DeviceSetup dev;
    const int32_t st = setup_current_device(device, &dev);
    if (st != OD_OK) return st;

    // A context on the stack, only to hand the launcher its parameters; nothing in
    // it is allocated or freed, and the scratch pointer is the static array.
    od_ctx c = {};
    c.device = device;
    c.v_p = target_vocab;
    c.max_batch = B;
    c.max_k = K_max;
    c.sm_count = dev.sm_count;
    c.d_partials = dev.partials;
    c.opt_pdl = 1;
    c.verify_early = false;     // nothing is known about the launch in front: wait before reading
    if (od_launch_verify(&c, B, K_max, logits, logit_dtype, row_stride, seq_stride, tgt_ids, q_prime,
                         span_len, m, temperature, seed, step, row_max, row_sum, p_sel, ratio,
                         n_accepted, n_draft_accepted, verify_flags, (cudaStream_t)stream) != cudaSuccess)
        return OD_ERR_CUDA;
    return OD_OK;
}
