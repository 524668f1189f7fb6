// Step 1: translation of the draft proposal into the target vocabulary
// (Section 3.1, Eq. (1); Algorithm 1, translation line).
//
// One thread block per sequence, one warp per proposal offset. Warp s probes
// the n-gram cache for the runs of length 4, 3, 2 that start at offset s: the
// cache is an open-addressing table of 32-slot groups, a probe reads one group
// with one coalesced 256-byte load (lane <-> slot) and resolves it with two
// ballots (key match / empty slot). The first probes of the three lengths are
// issued together, each with the values of its group, so their latencies overlap
// and a hit in the first group costs one memory round trip. After a block barrier one thread
// walks the proposal left to right, longest hit first, then the direct map,
// and writes the mapped proposal. Integer work throughout, except the product
// of at most four fp32 draft probabilities.
#include "od_common.cuh"

namespace {

// Resolves a lookup whose first group g is already loaded (keys in k_lane, values in
// v_lane): the slot that holds `key` and its value, or -1. Walks at most ngroups groups,
// so it ends on any table contents.
__device__ __forceinline__ int32_t probe_continue(const uint64_t *__restrict__ keys, const int32_t *__restrict__ vals,
                                                  uint64_t ngroups, uint64_t key, uint64_t g,
                                                  uint64_t k_lane, int32_t v_lane, int lane, int32_t *value)
{
    for (uint64_t step = 0; step < ngroups; ++step) {
        unsigned match = __ballot_sync(0xFFFFFFFFu, k_lane == key);
        if (match) {
            const int src = __ffs(match) - 1;
            *value = __shfl_sync(0xFFFFFFFFu, v_lane, src);
            return (int32_t)(g * OD_GROUP + src);
        }
        unsigned empty = __ballot_sync(0xFFFFFFFFu, k_lane == 0ULL);
        if (empty) return -1;
        g = (g + 1) & (ngroups - 1);
        k_lane = __ldg(keys + g * OD_GROUP + lane);
        v_lane = __ldcg(vals + g * OD_GROUP + lane);
    }
    return -1;
}

__global__ void __launch_bounds__(OD_MAX_K *OD_WARP)
od_map_kernel(int32_t B, int32_t K_max, int32_t v_q, const int32_t *__restrict__ draft_ids,
              const int32_t *__restrict__ draft_len, const float *__restrict__ q_sel,
              const int32_t *__restrict__ vocab_map, const uint64_t *__restrict__ keys,
              const int32_t *__restrict__ vals, int64_t cap, int32_t *__restrict__ tgt_ids,
              float *__restrict__ q_prime, int32_t *__restrict__ span_start,
              int32_t *__restrict__ span_len, int32_t *__restrict__ m_out,
              uint8_t *__restrict__ tail_kind, uint32_t *__restrict__ counters,
              uint32_t *__restrict__ stamp, uint32_t *__restrict__ freq, uint32_t clock, int32_t early)
{
    __shared__ int32_t s_ids[OD_MAX_K];
    __shared__ int32_t s_hit[OD_MAX_K][OD_NGRAM_MAX + 1];   // [offset][length] -> target or -1
    __shared__ int32_t s_slot[OD_MAX_K][OD_NGRAM_MAX + 1];  // the table slot of that hit
    __shared__ int32_t s_direct[OD_MAX_K];                  // direct map of the id at each offset, or -1
    __shared__ float s_q[OD_MAX_K];                         // q(d) of each offset

    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // The proposal itself (ids, length, probabilities) is the caller's input. Where the
    // caller has promised that it was complete before the launch in front of this one was
    // enqueued (early bit 0), it is requested before the wait. The n-gram table and the
    // vocabulary map belong to the context: unless a kernel that writes the table was
    // launched on this context since the last translation kernel (early bit 1 clear), the
    // probes run before the wait as well, and only the serial walk, which writes, is left
    // for after it. Inside od_step (early bit 2) the next kernel is the streaming pass, which
    // starts on logit rows 0 before its own wait (inputs under the same promise) and releases
    // ITS successor only after that wait: it is released at once, so that rows 0 stream under
    // the tail of the step in front.
    int K = 0;
    int32_t my_id = -1;
    float my_q = 0.f;
    const bool early_proposal = (early & 1) != 0, early_table = (early & 2) != 0, early_release = (early & 4) != 0;
    auto load_proposal = [&]() {
        K = draft_len[b];
        if (threadIdx.x < K_max) my_id = draft_ids[(size_t)b * K_max + threadIdx.x];
        if (lane == 0 && warp < K_max) my_q = q_sel[(size_t)b * K_max + warp];
    };
    auto probe = [&]() {
        K = K < 0 ? 0 : (K > K_max ? K_max : K);
        if (threadIdx.x < K_max) s_ids[threadIdx.x] = my_id;
        __syncthreads();

        const int s = warp;
        if (s < K) {
            // what the serial walk below would otherwise fetch one position at a time
            if (lane == 0) {
                const int32_t id = s_ids[s];
                s_direct[s] = (id >= 0 && id < v_q) ? __ldg(vocab_map + id) : -1;
                s_q[s] = my_q;
            }
            int32_t hit[OD_NGRAM_MAX + 1] = {-1, -1, -1, -1, -1};
            int32_t slot[OD_NGRAM_MAX + 1] = {-1, -1, -1, -1, -1};
            if (cap > 0) {
                const uint64_t ngroups = (uint64_t)cap / OD_GROUP;
                uint64_t key[OD_NGRAM_MAX + 1], grp[OD_NGRAM_MAX + 1], kl[OD_NGRAM_MAX + 1];
                int32_t vl[OD_NGRAM_MAX + 1];
                bool valid[OD_NGRAM_MAX + 1];
                // ids of a run must lie in the draft vocabulary; the run must fit
                bool ok = true;
                uint64_t k = 0;
#pragma unroll
                for (int L = 1; L <= OD_NGRAM_MAX; ++L) {
                    int32_t id = (s + L - 1 < K) ? s_ids[s + L - 1] : -1;
                    ok = ok && (s + L <= K) && id >= 0 && id < v_q;
                    k |= (uint64_t)(uint32_t)(id + 1) << (16 * (L - 1));
                    valid[L] = ok && L >= 2;
                    key[L] = k;
                    grp[L] = od_hash64(k) & (ngroups - 1);
                }
#pragma unroll
                for (int L = 2; L <= OD_NGRAM_MAX; ++L) {
                    kl[L] = valid[L] ? __ldg(keys + grp[L] * OD_GROUP + lane) : 0ULL;
                    // the values of the group come with its keys, so a hit costs one round trip
                    // (a concurrent batch insert writes an entry's value last: read it past L1)
                    vl[L] = valid[L] ? __ldcg(vals + grp[L] * OD_GROUP + lane) : -1;
                }
#pragma unroll
                for (int L = 2; L <= OD_NGRAM_MAX; ++L)
                    if (valid[L]) {
                        int32_t value = -1;
                        slot[L] = probe_continue(keys, vals, ngroups, key[L], grp[L], kl[L], vl[L], lane, &value);
                        // an entry whose value is not set yet does not exist
                        if (slot[L] >= 0) hit[L] = value;
                    }
            }
            if (lane == 0) {
#pragma unroll
                for (int L = 2; L <= OD_NGRAM_MAX; ++L) { s_hit[s][L] = hit[L]; s_slot[s][L] = slot[L]; }
            }
        }
    };
    if (early_release) asm volatile("griddepcontrol.launch_dependents;");
    if (early_proposal && b < B) {
        load_proposal();
        if (early_table) probe();
    }

    // under programmatic dependent launch: wait for everything earlier in the
    // stream first, only then (no promise) let the verification kernel start its prefetch
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!early_release) asm volatile("griddepcontrol.launch_dependents;");

    if (b >= B) return;
    if (!early_proposal) load_proposal();
    if (!(early_proposal && early_table)) probe();
    __syncthreads();

    if (threadIdx.x == 0) {
        const size_t o = (size_t)b * K_max;
        int pos = 0, m = 0;
        uint32_t hits = 0, invalid = 0;
        uint8_t tail = OD_TAIL_COMPLETE;
        while (pos < K) {
            int L = 0;
            int32_t t = -1;
            for (int len = OD_NGRAM_MAX; len >= 2; --len)
                if (pos + len <= K && s_hit[pos][len] >= 0) { L = len; t = s_hit[pos][len]; break; }
            if (L) {
                float prod = s_q[pos];
                for (int j = 1; j < L; ++j) prod *= s_q[pos + j];
                tgt_ids[o + m] = t; q_prime[o + m] = prod;
                span_start[o + m] = pos; span_len[o + m] = L;
                if (stamp) {                                // an access: recency and frequency of the entry
                    atomicMax(stamp + s_slot[pos][L], clock);
                    atomicAdd(freq + s_slot[pos][L], 1u);
                }
                ++m; pos += L; ++hits;
                continue;
            }
            const int32_t id = s_ids[pos];
            const bool in_vocab = id >= 0 && id < v_q;
            if (!in_vocab) ++invalid;
            const int32_t direct = s_direct[pos];
            if (direct >= 0) {
                tgt_ids[o + m] = direct; q_prime[o + m] = s_q[pos];
                span_start[o + m] = pos; span_len[o + m] = 1;
                ++m; ++pos;
            } else {
                span_start[o + m] = pos; span_len[o + m] = 1;
                tail = OD_TAIL_UNMAPPED_STOP;
                break;
            }
        }
        m_out[b] = m;
        tail_kind[b] = tail;
        if (counters) {
            if (hits) atomicAdd(counters + OD_CNT_CACHE_HITS, hits);
            if (tail == OD_TAIL_UNMAPPED_STOP) atomicAdd(counters + OD_CNT_UNMAPPED_STOPS, 1u);
            if (invalid) atomicAdd(counters + OD_CNT_INVALID_IDS, invalid);
            if (m) atomicAdd(counters + OD_CNT_MAPPED_TOKENS, (uint32_t)m);
        }
    }
}

}  // namespace

cudaError_t od_launch_map(od_ctx *c, int32_t B, int32_t K_max, const int32_t *draft_ids,
                          const int32_t *draft_len, const float *q_sel, int32_t *tgt_ids,
                          float *q_prime, int32_t *span_start, int32_t *span_len, int32_t *m,
                          uint8_t *tail_kind, uint32_t *counters, bool early, bool release_early,
                          cudaStream_t s)
{
    if (B == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)B);
    cfg.blockDim = dim3((unsigned)(K_max * OD_WARP));
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->opt_pdl ? 1 : 0;
    c->last_was_map = true;
    // A kernel that writes the table (insert, trim) may be the launch in front of this one: then
    // the probes stay behind the wait. A translation kernel releases its successor after its
    // wait, or (inside od_step) that successor is the streaming pass, which does: either way
    // every later translation kernel starts after those writers are done.
    const int32_t early_bits = early && c->opt_pdl ? (c->table_written ? 1 : 3) | (release_early ? 4 : 0) : 0;
    c->table_written = false;
    return cudaLaunchKernelEx(&cfg, od_map_kernel, B, K_max, c->v_q, draft_ids, draft_len, q_sel,
                              (const int32_t *)c->d_vocab_map, (const uint64_t *)c->d_keys,
                              (const int32_t *)c->d_vals, c->cap, tgt_ids, q_prime, span_start,
                              span_len, m, tail_kind, counters, c->dyn ? c->d_stamp : (uint32_t *)nullptr,
                              c->dyn ? c->d_freq : (uint32_t *)nullptr, c->clock, early_bits);
}
