// Online n-gram cache: insertion of unseen n-grams (Algorithm 1, cache-update line)
// and bounded size with LRU / LFU eviction (App. D.5, cache scalability).
//
// The table is the open-addressing table od_map_proposals probes (groups of 32
// slots), with three more words per slot: clock of the last access, access
// frequency, clock of insertion. Nothing is ever deleted in place, so lookups stay
// lock-free and simple; eviction rebuilds the table.
//   insert  one thread per candidate claims the first empty slot of its probe
//           sequence with a compare-and-swap on the key; candidates of one batch
//           that carry the same run settle on the one with the lowest index
//           (atomicMin on a claim word) and that one writes the value last, so a
//           concurrent or later lookup sees either nothing or the whole entry, and
//           the result does not depend on thread timing.
//   trim    with k = size - max_entries > 0 entries too many, the k entries that
//           come first in the order (inserted at the current clock?, score, run key)
//           are dropped, score = last-access clock (LRU) or frequency (LFU). The
//           k-th smallest is found by a most-significant-digit radix select over the
//           104-bit order key (13 passes of a histogram kernel whose last block to
//           finish picks the digit, no sorting); then the survivors are re-inserted
//           into the spare table, which becomes the table. No kernel waits for another.
#include <string.h>
#include <utility>
#include <vector>

#include "od_common.cuh"

namespace {

struct TrimState {
    unsigned int size;          // live entries of the current table
    unsigned int k;             // entries to drop in this trim
    unsigned int k_rem;         // rank still to resolve among the entries matching the prefix
    unsigned int pad;
    unsigned long long pre_hi, pre_lo, mask_hi, mask_lo;   // decided digits of the k-th order key
    unsigned int hist[256];
    unsigned int invalid;       // malformed candidates seen by od_cache_insert
    unsigned int ticket;        // blocks of the running histogram pass that are done
};

constexpr int PASSES = 13;      // 5 bytes of (new?, score), 8 bytes of the run key

// order key of a live entry: hi = (inserted at the current clock) << 32 | score, lo = run key
__device__ __forceinline__ void order_key(int policy, unsigned int clock, unsigned long long key,
                                          unsigned int stamp, unsigned int freq, unsigned int born,
                                          unsigned long long &hi, unsigned long long &lo)
{
    hi = ((unsigned long long)(born == clock ? 1u : 0u) << 32) | (policy == 0 ? stamp : freq);
    lo = key;
}

__device__ __forceinline__ unsigned int digit_of(int pass, unsigned long long hi, unsigned long long lo)
{
    return pass < 5 ? (unsigned int)(hi >> (8 * (4 - pass))) & 0xFFu
                    : (unsigned int)(lo >> (8 * (12 - pass))) & 0xFFu;
}

__global__ void insert_claim_kernel(int32_t N, int32_t v_q, int32_t v_p, const int32_t *__restrict__ runs,
                                    const int32_t *__restrict__ len, const int32_t *__restrict__ target,
                                    unsigned long long *keys, const int32_t *vals, int64_t cap,
                                    unsigned int *owner, int32_t *cand_slot, TrimState *st)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    cand_slot[i] = -1;
    const int L = len[i];
    bool ok = L >= 2 && L <= OD_NGRAM_MAX && target[i] >= 0 && target[i] < v_p;
    int32_t ids[OD_NGRAM_MAX];
    for (int j = 0; j < OD_NGRAM_MAX; ++j) {
        ids[j] = j < L && ok ? runs[(size_t)i * OD_NGRAM_MAX + j] : 0;
        if (j < L && ok && (ids[j] < 0 || ids[j] >= v_q)) ok = false;
    }
    if (!ok) { atomicAdd(&st->invalid, 1u); return; }
    const unsigned long long key = od_pack_run(ids, L);
    const uint64_t ngroups = (uint64_t)cap / OD_GROUP;
    uint64_t g = od_hash64(key) & (ngroups - 1);
    for (uint64_t step = 0; step < ngroups; ++step) {       // bounded: ends on any table contents
        for (int s = 0; s < OD_GROUP; ++s) {
            const int64_t slot = (int64_t)(g * OD_GROUP + s);
            unsigned long long cur = keys[slot];
            if (cur == 0ull) cur = atomicCAS(keys + slot, 0ull, key);   // 0 again: the slot is ours
            if (cur == 0ull || cur == key) {
                // an entry with a value was there before this batch: nothing to add
                if (((volatile const int32_t *)vals)[slot] < 0) {
                    atomicMin(owner + slot, (unsigned int)i);
                    cand_slot[i] = (int32_t)slot;
                }
                return;
            }
        }
        g = (g + 1) & (ngroups - 1);
    }
}

__global__ void insert_commit_kernel(int32_t N, const int32_t *__restrict__ target, int32_t *vals,
                                     unsigned int *stamp, unsigned int *freq, unsigned int *born,
                                     unsigned int *owner, const int32_t *__restrict__ cand_slot,
                                     unsigned int clock, TrimState *st)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int32_t slot = cand_slot[i];
    if (slot < 0 || owner[slot] != (unsigned int)i) return; // a candidate with a lower index carries this run
    stamp[slot] = clock; freq[slot] = 1u; born[slot] = clock;
    __threadfence();
    vals[slot] = target[i];                                  // the entry exists from here on
    owner[slot] = 0xFFFFFFFFu;
    atomicAdd(&st->size, 1u);
}

__global__ void trim_begin_kernel(TrimState *st, unsigned int max_entries)
{
    st->k = st->size > max_entries ? st->size - max_entries : 0u;
    st->k_rem = st->k;
    st->pre_hi = st->pre_lo = st->mask_hi = st->mask_lo = 0ull;
    for (int i = 0; i < 256; ++i) st->hist[i] = 0u;
    st->ticket = 0u;
}

__global__ void trim_hist_kernel(int pass, int policy, unsigned int clock, const unsigned long long *keys,
                                 const int32_t *vals, const unsigned int *stamp, const unsigned int *freq,
                                 const unsigned int *born, int64_t cap, TrimState *st)
{
    __shared__ unsigned int s_hist[256];
    if (st->k == 0u) return;                                 // nothing to drop: every block leaves
    s_hist[threadIdx.x] = 0u;
    __syncthreads();
    const unsigned long long pre_hi = st->pre_hi, pre_lo = st->pre_lo, m_hi = st->mask_hi, m_lo = st->mask_lo;
    // four consecutive slots per thread and iteration, every load issued before the first
    // use: the pass is a chain of memory round trips otherwise (the table sits in L2)
    const unsigned int *score = policy == 0 ? stamp : freq;
    for (int64_t slot = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; slot < cap;
         slot += (int64_t)gridDim.x * blockDim.x * 4) {
        const ulonglong2 k01 = __ldg((const ulonglong2 *)(keys + slot));
        const ulonglong2 k23 = __ldg((const ulonglong2 *)(keys + slot) + 1);
        const int4 v4 = __ldg((const int4 *)(vals + slot));
        const uint4 s4 = __ldg((const uint4 *)(score + slot));
        const uint4 b4 = __ldg((const uint4 *)(born + slot));
        const unsigned long long kk[4] = {k01.x, k01.y, k23.x, k23.y};
        const int vv[4] = {v4.x, v4.y, v4.z, v4.w};
        const unsigned int ss[4] = {s4.x, s4.y, s4.z, s4.w};
        const unsigned int bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (kk[e] == 0ull || vv[e] < 0) continue;
            const unsigned long long hi = ((unsigned long long)(bb[e] == clock ? 1u : 0u) << 32) | ss[e], lo = kk[e];
            if ((hi & m_hi) == pre_hi && (lo & m_lo) == pre_lo) {
                // scores are heavily tied (most digits are equal across the table): one
                // shared-memory add per distinct digit of the warp, not one per entry
                const unsigned int d = digit_of(pass, hi, lo);
                const unsigned int peers = __match_any_sync(__activemask(), d);
                if ((int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&s_hist[d], (unsigned int)__popc(peers));
            }
        }
    }
    __syncthreads();
    if (s_hist[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], s_hist[threadIdx.x]);

    // The block that finishes last picks the digit in which the running count reaches
    // k_rem (no second launch per pass): the barrier orders this block's adds before
    // thread 0's fence and ticket; the last block fences again before it reads.
    __shared__ unsigned int s_last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&st->ticket, 1u) == gridDim.x - 1 ? 1u : 0u;
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    s_hist[threadIdx.x] = __ldcg(&st->hist[threadIdx.x]);
    __syncthreads();
    if (threadIdx.x < 32) {
        // warp 0: lane l owns bins 8l .. 8l+7; the first bin at which the running count reaches k_rem
        const int lane = threadIdx.x;
        const unsigned int k_rem = st->k_rem;
        unsigned int mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) mine += s_hist[lane * 8 + i];
        unsigned int inc = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int t = __shfl_up_sync(0xFFFFFFFFu, inc, off);
            if (lane >= off) inc += t;
        }
        const unsigned int reach = __ballot_sync(0xFFFFFFFFu, inc >= k_rem);
        const int owner = reach ? __ffs(reach) - 1 : 31;
        unsigned int run = inc - mine, d = 255;
        if (lane == owner) {
            for (int i = 0; i < 8; ++i) {
                if (run + s_hist[lane * 8 + i] >= k_rem) { d = lane * 8 + i; break; }
                run += s_hist[lane * 8 + i];
            }
            if (d == 255u && !reach) run = inc;             // counts fell short: everything below the last bin
        }
        d = __shfl_sync(0xFFFFFFFFu, d, owner);
        run = __shfl_sync(0xFFFFFFFFu, run, owner);
        if (lane == 0) {
            st->k_rem = k_rem - run;
            if (pass < 5) {
                st->pre_hi |= (unsigned long long)d << (8 * (4 - pass));
                st->mask_hi |= 0xFFull << (8 * (4 - pass));
            } else {
                st->pre_lo |= (unsigned long long)d << (8 * (12 - pass));
                st->mask_lo |= 0xFFull << (8 * (12 - pass));
            }
            st->ticket = 0u;
        }
    }
    st->hist[threadIdx.x] = 0u;
}

__global__ void table_clear_kernel(unsigned long long *keys, int32_t *vals, unsigned int *stamp,
                                   unsigned int *freq, unsigned int *born, int64_t cap)
{
    for (int64_t slot = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; slot < cap;
         slot += (int64_t)gridDim.x * blockDim.x) {
        keys[slot] = 0ull; vals[slot] = -1; stamp[slot] = 0u; freq[slot] = 0u; born[slot] = 0u;
    }
}

// survivors of the old table go into the (cleared) new one; run keys are distinct, so
// a plain compare-and-swap placement is deterministic as a set
__global__ void trim_rebuild_kernel(int policy, unsigned int clock, const unsigned long long *keys,
                                    const int32_t *vals, const unsigned int *stamp, const unsigned int *freq,
                                    const unsigned int *born, unsigned long long *nkeys, int32_t *nvals,
                                    unsigned int *nstamp, unsigned int *nfreq, unsigned int *nborn,
                                    int64_t cap, const TrimState *st)
{
    const unsigned int k = st->k;
    const unsigned long long thr_hi = st->pre_hi, thr_lo = st->pre_lo;
    const uint64_t ngroups = (uint64_t)cap / OD_GROUP;
    for (int64_t slot4 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; slot4 < cap;
         slot4 += (int64_t)gridDim.x * blockDim.x * 4) {
        // as in the histogram pass: four slots, all loads first
        const ulonglong2 k01 = __ldg((const ulonglong2 *)(keys + slot4));
        const ulonglong2 k23 = __ldg((const ulonglong2 *)(keys + slot4) + 1);
        const int4 v4 = __ldg((const int4 *)(vals + slot4));
        const uint4 s4 = __ldg((const uint4 *)(stamp + slot4));
        const uint4 f4 = __ldg((const uint4 *)(freq + slot4));
        const uint4 b4 = __ldg((const uint4 *)(born + slot4));
        const unsigned long long kk[4] = {k01.x, k01.y, k23.x, k23.y};
        const int vv[4] = {v4.x, v4.y, v4.z, v4.w};
        const unsigned int ss[4] = {s4.x, s4.y, s4.z, s4.w};
        const unsigned int ff[4] = {f4.x, f4.y, f4.z, f4.w};
        const unsigned int bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const unsigned long long key = kk[e];
            if (key == 0ull || vv[e] < 0) continue;
            if (k > 0u) {
                unsigned long long hi, lo;
                order_key(policy, clock, key, ss[e], ff[e], bb[e], hi, lo);
                if (hi < thr_hi || (hi == thr_hi && lo <= thr_lo)) continue;   // among the k first: dropped
            }
            uint64_t g = od_hash64(key) & (ngroups - 1);
            bool placed = false;
            for (uint64_t step = 0; step < ngroups && !placed; ++step) {
                for (int sl = 0; sl < OD_GROUP; ++sl) {
                    const int64_t ns = (int64_t)(g * OD_GROUP + sl);
                    if (nkeys[ns] == 0ull && atomicCAS(nkeys + ns, 0ull, key) == 0ull) {
                        nvals[ns] = vv[e]; nstamp[ns] = ss[e]; nfreq[ns] = ff[e]; nborn[ns] = bb[e];
                        placed = true;
                        break;
                    }
                }
                g = (g + 1) & (ngroups - 1);
            }
        }
    }
}

__global__ void trim_end_kernel(TrimState *st) { st->size -= st->k; st->k = 0u; }

#define OD_CUDA(call)                                  \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) return OD_ERR_CUDA;    \
    } while (0)

struct Guard {
    int prev; bool ok;
    explicit Guard(int dev) : prev(-1), ok(false) { if (cudaGetDevice(&prev) == cudaSuccess) ok = cudaSetDevice(dev) == cudaSuccess; }
    ~Guard() { if (prev >= 0) cudaSetDevice(prev); }
};

template <typename T>
int32_t alloc_zero(T **p, size_t n)
{
    *p = nullptr;
    cudaError_t e = cudaMalloc((void **)p, (n ? n : 1) * sizeof(T));
    if (e == cudaErrorMemoryAllocation) return OD_ERR_NOMEM;
    if (e != cudaSuccess) return OD_ERR_CUDA;
    return cudaMemset(*p, 0, (n ? n : 1) * sizeof(T)) == cudaSuccess ? OD_OK : OD_ERR_CUDA;
}

}  // namespace

void od_cache_free_dynamic(od_ctx *c)
{
    void *ptrs[] = {c->d_stamp, c->d_freq, c->d_born, c->d_keys2, c->d_vals2, c->d_stamp2, c->d_freq2,
                    c->d_born2, c->d_owner, c->d_cand_slot, c->d_trim};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    c->d_stamp = c->d_freq = c->d_born = c->d_stamp2 = c->d_freq2 = c->d_born2 = c->d_owner = nullptr;
    c->d_keys2 = nullptr; c->d_vals2 = nullptr; c->d_cand_slot = nullptr; c->d_trim = nullptr;
    c->dyn = false;
}

extern "C" {

int32_t od_cache_configure(od_ctx *c, int64_t max_entries, int32_t policy, int32_t max_insert)
{
    if (!c || max_entries < 1 || max_entries > ((int64_t)1 << 28) || max_insert < 1 ||
        max_insert > (1 << 24) || (policy != 0 && policy != 1))
        return OD_ERR_INVALID_ARG;
    if (c->v_q > 65535) return OD_ERR_UNSUPPORTED;           // a run packs 16 bits per id
    Guard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(cudaDeviceSynchronize());
    od_cache_free_dynamic(c);
    if (c->d_keys) { cudaFree(c->d_keys); c->d_keys = nullptr; }
    if (c->d_vals) { cudaFree(c->d_vals); c->d_vals = nullptr; }
    c->cap = 0;
    int64_t cap = 64;
    while (cap < 2 * (max_entries + max_insert)) cap <<= 1;  // load stays under 1/2 even before a trim
    int32_t st = alloc_zero(&c->d_keys, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_vals, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_stamp, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_freq, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_born, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_keys2, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_vals2, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_stamp2, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_freq2, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_born2, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_owner, (size_t)cap);
    if (st == OD_OK) st = alloc_zero(&c->d_cand_slot, (size_t)max_insert);
    TrimState *ts = nullptr;
    if (st == OD_OK) st = alloc_zero(&ts, 1);
    c->d_trim = ts;
    if (st != OD_OK) { od_cache_free_dynamic(c); return st; }
    OD_CUDA(cudaMemset(c->d_vals, 0xFF, (size_t)cap * sizeof(int32_t)));    // -1: no value
    OD_CUDA(cudaMemset(c->d_vals2, 0xFF, (size_t)cap * sizeof(int32_t)));
    OD_CUDA(cudaMemset(c->d_owner, 0xFF, (size_t)cap * sizeof(uint32_t)));
    c->cap = cap;
    c->dyn = true; c->dyn_policy = policy; c->dyn_max = max_entries; c->dyn_max_insert = max_insert;
    c->clock = 0;
    return OD_OK;
}

int32_t od_cache_set_clock(od_ctx *c, uint32_t clock)
{
    if (!c) return OD_ERR_INVALID_ARG;
    if (!c->dyn) return OD_ERR_STATE;
    c->clock = clock;
    return OD_OK;
}

int32_t od_cache_insert(od_ctx *c, int32_t N, const int32_t *runs, const int32_t *len,
                        const int32_t *target, void *stream)
{
    if (!c || N < 0) return OD_ERR_INVALID_ARG;
    if (!c->dyn) return OD_ERR_STATE;
    if (N > c->dyn_max_insert) return OD_ERR_INVALID_ARG;
    if (N == 0) return OD_OK;
    if (!runs || !len || !target) return OD_ERR_INVALID_ARG;
    Guard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    c->last_was_map = false;
    const int threads = 128, blocks = (N + threads - 1) / threads;
    insert_claim_kernel<<<blocks, threads, 0, s>>>(N, c->v_q, c->v_p, runs, len, target,
                                                   (unsigned long long *)c->d_keys, c->d_vals, c->cap,
                                                   c->d_owner, c->d_cand_slot, (TrimState *)c->d_trim);
    insert_commit_kernel<<<blocks, threads, 0, s>>>(N, target, c->d_vals, c->d_stamp, c->d_freq, c->d_born,
                                                    c->d_owner, c->d_cand_slot, c->clock,
                                                    (TrimState *)c->d_trim);
    OD_CUDA(cudaGetLastError());
    return OD_OK;
}

int32_t od_cache_trim(od_ctx *c, void *stream)
{
    if (!c) return OD_ERR_INVALID_ARG;
    if (!c->dyn) return OD_ERR_STATE;
    Guard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    c->last_was_map = false;
    TrimState *st = (TrimState *)c->d_trim;
    const int grid = c->sm_count * 4;
    trim_begin_kernel<<<1, 1, 0, s>>>(st, (unsigned int)c->dyn_max);
    for (int pass = 0; pass < PASSES; ++pass) {
        trim_hist_kernel<<<grid, 256, 0, s>>>(pass, c->dyn_policy, c->clock, (const unsigned long long *)c->d_keys,
                                              c->d_vals, c->d_stamp, c->d_freq, c->d_born, c->cap, st);
    }
    table_clear_kernel<<<grid, 256, 0, s>>>((unsigned long long *)c->d_keys2, c->d_vals2, c->d_stamp2,
                                            c->d_freq2, c->d_born2, c->cap);
    trim_rebuild_kernel<<<grid, 256, 0, s>>>(c->dyn_policy, c->clock, (const unsigned long long *)c->d_keys,
                                             c->d_vals, c->d_stamp, c->d_freq, c->d_born,
                                             (unsigned long long *)c->d_keys2, c->d_vals2, c->d_stamp2,
                                             c->d_freq2, c->d_born2, c->cap, st);
    trim_end_kernel<<<1, 1, 0, s>>>(st);
    OD_CUDA(cudaGetLastError());
    // the rebuilt table is the table for every call enqueued from now on
    std::swap(c->d_keys, c->d_keys2); std::swap(c->d_vals, c->d_vals2);
    std::swap(c->d_stamp, c->d_stamp2); std::swap(c->d_freq, c->d_freq2); std::swap(c->d_born, c->d_born2);
    return OD_OK;
}

int32_t od_cache_dump(od_ctx *c, int64_t max_out, int32_t *runs, int32_t *len, int32_t *target,
                      uint32_t *stamp, uint32_t *freq, int64_t *n_out)
{
    if (!c || !n_out || max_out < 0) return OD_ERR_INVALID_ARG;
    if (!c->dyn) return OD_ERR_STATE;
    Guard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(cudaDeviceSynchronize());
    const size_t cap = (size_t)c->cap;
    std::vector<uint64_t> keys(cap);
    std::vector<int32_t> vals(cap);
    std::vector<uint32_t> st(cap), fr(cap);
    OD_CUDA(cudaMemcpy(keys.data(), c->d_keys, cap * 8, cudaMemcpyDeviceToHost));
    OD_CUDA(cudaMemcpy(vals.data(), c->d_vals, cap * 4, cudaMemcpyDeviceToHost));
    OD_CUDA(cudaMemcpy(st.data(), c->d_stamp, cap * 4, cudaMemcpyDeviceToHost));
    OD_CUDA(cudaMemcpy(fr.data(), c->d_freq, cap * 4, cudaMemcpyDeviceToHost));
    int64_t n = 0;
    for (size_t s = 0; s < cap; ++s) {
        if (keys[s] == 0 || vals[s] < 0) continue;
        if (n < max_out && runs && len && target) {
            int L = 0;
            for (int j = 0; j < OD_NGRAM_MAX; ++j) {
                const uint32_t f = (uint32_t)(keys[s] >> (16 * j)) & 0xFFFFu;
                runs[n * OD_NGRAM_MAX + j] = f ? (int32_t)f - 1 : -1;
                if (f) L = j + 1;
            }
            len[n] = L; target[n] = vals[s];
            if (stamp) stamp[n] = st[s];
            if (freq) freq[n] = fr[s];
        }
        ++n;
    }
    *n_out = n;
    return OD_OK;
}

}  // extern "C"
