// Step 2: temperature softmax statistics of the m_b + 1 target-logit rows,
// acceptance ratios and the accepted prefix (Algorithm 1, target-probability
// and rejection-sampling lines; acceptance ratio of Section 3.1).
//
// The kernel is a single streaming pass over the logits: every element is read
// from HBM exactly once with 128-bit loads. A row is cut into chunks; one
// thread block reduces one chunk to a (max, sum exp) pair: per thread a
// running pair whose maximum is refreshed once per 16-byte vector (one rescale
// per vector, not per element), then a fixed shuffle tree over the warp and
// over the block's warps. Blocks never wait on one another: a block publishes
// its pair, takes a ticket on the row's counter, and the block that draws the
// last ticket merges the row's pairs in chunk order, evaluates p(t_i), the
// ratio, the uniform and the accept bit; the last row of a sequence (a second
// ticket) turns the accept bits into the prefix length. Tickets and bit words
// are reset by their last user, so every launch starts from zeros.
//
// The reduction order is fixed (no floating-point atomics): results are
// bit-identical from run to run.
#include <float.h>

#include "od_common.cuh"

namespace {

struct VerifyArgs {
    const void *logits;
    int64_t row_stride, seq_stride;     // elements
    int32_t B, K_max, v_p;
    int32_t chunk_elems, chunks;
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
    float2 *partials;
    unsigned int *row_ticket, *seq_ticket, *seq_bits;
};

// running pair update with the 8 (bf16) or 4 (fp32) values of one vector
__device__ __forceinline__ void absorb(float &m, float &s, const float *x, int n, float scale)
{
    float vm = x[0];
#pragma unroll
    for (int i = 1; i < 8; ++i)
        if (i < n) vm = fmaxf(vm, x[i]);
    if (vm > m) {
        s *= od_ex2((m - vm) * scale);
        m = vm;
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (i < n) acc += od_ex2((x[i] - m) * scale);
    s += acc;
}

template <int DTYPE>
__device__ __forceinline__ void unpack(const uint4 &v, float *x)
{
    if (DTYPE == OD_BF16) {
        x[0] = od_bf16_lo(v.x); x[1] = od_bf16_hi(v.x);
        x[2] = od_bf16_lo(v.y); x[3] = od_bf16_hi(v.y);
        x[4] = od_bf16_lo(v.z); x[5] = od_bf16_hi(v.z);
        x[6] = od_bf16_lo(v.w); x[7] = od_bf16_hi(v.w);
    } else {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <int DTYPE>
__global__ void __launch_bounds__(OD_VERIFY_THREADS)
od_verify_kernel(const VerifyArgs a)
{
    constexpr int VEC = DTYPE == OD_BF16 ? 8 : 4;          // elements per 16 bytes
    constexpr int UNROLL = 4;
    const int b = blockIdx.z, r = blockIdx.y, c = blockIdx.x;
    int mb = a.m[b];
    mb = mb < 0 ? 0 : (mb > a.K_max ? a.K_max : mb);
    if (r > mb) return;                                     // rows above m_b are never touched

    const float T = a.temperature[b];
    const bool bad_T = !(T > 0.f);
    const float scale = bad_T ? 0.f : 1.4426950408889634f / T;   // log2(e)/T
    const size_t esz = DTYPE == OD_BF16 ? 2 : 4;
    const char *row = (const char *)a.logits + ((size_t)b * a.seq_stride + (size_t)r * a.row_stride) * esz;

    const int64_t lo = (int64_t)c * a.chunk_elems;
    int64_t hi = lo + a.chunk_elems;
    if (hi > a.v_p) hi = a.v_p;
    const int64_t nvec = (hi - lo) / VEC;                  // whole vectors in this chunk
    const uint4 *vp = (const uint4 *)(row + (size_t)lo * esz);

    float tm = -FLT_MAX, ts = 0.f;
    int64_t i = threadIdx.x;
    for (; i + (UNROLL - 1) * OD_VERIFY_THREADS < nvec; i += UNROLL * OD_VERIFY_THREADS) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream(vp + i + u * OD_VERIFY_THREADS);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            float x[8];
            unpack<DTYPE>(v[u], x);
            absorb(tm, ts, x, VEC, scale);
        }
    }
    for (; i < nvec; i += OD_VERIFY_THREADS) {
        float x[8];
        unpack<DTYPE>(ld_stream(vp + i), x);
        absorb(tm, ts, x, VEC, scale);
    }
    // ragged tail of the row (v_p not a multiple of the vector width)
    {
        const int64_t t0 = lo + nvec * VEC + threadIdx.x;
        if (t0 < hi) {
            float x[8];
            x[0] = od_load_logit<DTYPE>(row, t0);
            absorb(tm, ts, x, 1, scale);
        }
    }

    // block reduction: shuffle tree inside the warp, then over the warps
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        float m2 = __shfl_xor_sync(0xFFFFFFFFu, tm, off);
        float s2 = __shfl_xor_sync(0xFFFFFFFFu, ts, off);
        od_pair_merge(tm, ts, m2, s2, scale);
    }
    __shared__ float sm_m[OD_VERIFY_THREADS / 32], sm_s[OD_VERIFY_THREADS / 32];
    __shared__ unsigned int s_ticket;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { sm_m[warp] = tm; sm_s[warp] = ts; }
    __syncthreads();

    const int row_slot = b * (a.K_max + 1) + r;
    if (threadIdx.x == 0) {
        float bm = sm_m[0], bs = sm_s[0];
        for (int w = 1; w < OD_VERIFY_THREADS / 32; ++w) od_pair_merge(bm, bs, sm_m[w], sm_s[w], scale);
        a.partials[(size_t)row_slot * a.chunks + c] = make_float2(bm, bs);
        __threadfence();
        s_ticket = atomicAdd(a.row_ticket + row_slot, 1u);
    }
    __syncthreads();
    if (s_ticket != (unsigned)(a.chunks - 1)) return;       // not the last block of this row

    // ---- last block of the row: merge the chunks in order, decide position r ----
    if (threadIdx.x != 0) return;
    __threadfence();
    a.row_ticket[row_slot] = 0;
    float M, S;
    {
        const volatile float2 *pp = (const volatile float2 *)(a.partials + (size_t)row_slot * a.chunks);
        M = pp[0].x; S = pp[0].y;
        for (int k = 1; k < a.chunks; ++k) od_pair_merge(M, S, pp[k].x, pp[k].y, scale);
    }
    a.row_max[row_slot] = M;
    a.row_sum[row_slot] = S;
    unsigned int bits = 0;
    if (!(S > 0.f) || !(S <= FLT_MAX)) atomicOr(a.seq_bits + 2 * b + 1, 1u);   // not finite and positive
    if (r < mb) {
        const size_t o = (size_t)b * a.K_max + r;
        const int32_t t = a.tgt_ids[o];
        float p = 0.f;
        if (t >= 0 && t < a.v_p) p = od_ex2((od_load_logit<DTYPE>(row, t) - M) * scale) / S;
        const float q = a.q_prime[o];
        const float ra = (q <= p) ? 1.f : p / q;
        const float u = od_uniform(a.seed[b], a.step, (uint32_t)r, 0u);
        a.p_sel[o] = p;
        a.ratio[o] = ra;
        if (u < ra) bits |= 1u << r;
        if (fabsf(u - ra) <= OD_TAU_ACCEPT) bits |= 1u << (16 + r);
    }
    if (bits) atomicOr(a.seq_bits + 2 * b, bits);
    __threadfence();
    const unsigned int st = atomicAdd(a.seq_ticket + b, 1u);
    if (st != (unsigned)mb) return;                         // rows 0..m_b: m_b + 1 tickets

    // ---- last row of the sequence: accepted prefix ----
    __threadfence();
    const unsigned int all = atomicExch(a.seq_bits + 2 * b, 0u);
    const unsigned int misc = atomicExch(a.seq_bits + 2 * b + 1, 0u);
    a.seq_ticket[b] = 0;
    int n = 0;
    while (n < mb && (all >> n & 1u)) ++n;
    int nd = 0;
    for (int k = 0; k < n; ++k) nd += a.span_len[(size_t)b * a.K_max + k];
    uint32_t f = (all >> 16) & OD_VF_BOUNDARY_MASK;
    if (misc & 1u) f |= OD_VF_NONFINITE;
    if (bad_T) { f |= OD_VF_BAD_TEMPERATURE; n = 0; nd = 0; }
    a.n_accepted[b] = n;
    a.n_draft_accepted[b] = nd;
    a.flags[b] = f;
}

}  // namespace

cudaError_t od_launch_verify(od_ctx *c, int32_t B, int32_t K_max, const void *logits,
                             int32_t dtype, int64_t row_stride, int64_t seq_stride,
                             const int32_t *tgt_ids, const float *q_prime,
                             const int32_t *span_len, const int32_t *m,
                             const float *temperature, const uint64_t *seed, uint64_t step,
                             float *row_max, float *row_sum, float *p_sel, float *ratio,
                             int32_t *n_accepted, int32_t *n_draft_accepted,
                             uint32_t *flags, cudaStream_t s)
{
    if (B == 0) return cudaSuccess;
    const int64_t esz = dtype == OD_BF16 ? 2 : 4;
    const int64_t row_bytes = (int64_t)c->v_p * esz;
    const int64_t gran = 4096;                              // 256 threads x 16 bytes
    int64_t chunk_bytes = c->opt_verify_chunk_bytes;
    if (chunk_bytes <= 0) {
        // enough blocks to fill the machine several times over, chunks of 8..64 KB
        const int64_t rows = (int64_t)B * (K_max + 1);
        const int64_t want_blocks = (int64_t)c->sm_count * 16;
        int64_t per_row = (want_blocks + rows - 1) / rows;
        if (per_row < 1) per_row = 1;
        chunk_bytes = (row_bytes + per_row - 1) / per_row;
        if (chunk_bytes < 8192) chunk_bytes = 8192;
        if (chunk_bytes > 65536) chunk_bytes = 65536;
    }
    chunk_bytes = (chunk_bytes + gran - 1) / gran * gran;
    int64_t chunks = (row_bytes + chunk_bytes - 1) / chunk_bytes;
    if (chunks > c->max_chunks) {                           // scratch was sized for 4 KB chunks at most
        chunks = c->max_chunks;
        chunk_bytes = ((row_bytes + chunks - 1) / chunks + gran - 1) / gran * gran;
        chunks = (row_bytes + chunk_bytes - 1) / chunk_bytes;
    }
    VerifyArgs a;
    a.logits = logits; a.row_stride = row_stride; a.seq_stride = seq_stride;
    a.B = B; a.K_max = K_max; a.v_p = c->v_p;
    a.chunk_elems = (int32_t)(chunk_bytes / esz); a.chunks = (int32_t)chunks;
    a.tgt_ids = tgt_ids; a.q_prime = q_prime; a.span_len = span_len; a.m = m;
    a.temperature = temperature; a.seed = seed; a.step = step;
    a.row_max = row_max; a.row_sum = row_sum; a.p_sel = p_sel; a.ratio = ratio;
    a.n_accepted = n_accepted; a.n_draft_accepted = n_draft_accepted; a.flags = flags;
    a.partials = c->d_partials; a.row_ticket = c->d_row_ticket;
    a.seq_ticket = c->d_seq_ticket; a.seq_bits = c->d_seq_bits;
    dim3 grid((unsigned)chunks, (unsigned)(K_max + 1), (unsigned)B);
    c->info[0] = (int64_t)chunks * (K_max + 1) * B;
    c->info[1] = a.chunk_elems;
    if (dtype == OD_BF16)
        od_verify_kernel<OD_BF16><<<grid, OD_VERIFY_THREADS, 0, s>>>(a);
    else
        od_verify_kernel<OD_F32><<<grid, OD_VERIFY_THREADS, 0, s>>>(a);
    return cudaGetLastError();
}
