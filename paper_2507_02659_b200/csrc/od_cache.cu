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
//           are dropped, score = last-access clock (LRU) or frequency (LFU). One
//           pass over the table packs the live entries into a dense list (and clears
//           the spare table); the k-th smallest is found by a most-significant-digit
//           radix select over the 104-bit order key, 13 passes of a histogram kernel
//           over the CANDIDATES only: a pass copies the entries that still match the
//           decided prefix into the next list whenever that at least halves it, so
//           after the first digit that tells entries apart the passes are a few
//           hundred entries long. A pass is two dependent memory round trips: every
//           block works out the digit the pass before it decided from that pass's
//           256-bin histogram (redundantly, the same arithmetic everywhere), then
//           histograms its share of the next digit; no tickets, no fences, and a
//           digit of (new?, score) that is the same in every live entry costs no
//           histogram at all. Then the survivors are re-inserted from the dense list
//           into the spare table, which becomes the table. No kernel waits for another.
#include <stddef.h>
#include <string.h>
#include <utility>
#include <vector>

#include "od_common.cuh"

namespace {

constexpr int PASSES = 13;      // 5 bytes of (new?, score), 8 bytes of the run key

// What is known at the start of pass p: the digits before p of the k-th order key, the rank
// still to resolve among the candidates that match them, and where those candidates are.
struct SelState {
    unsigned long long pre_hi, pre_lo, mask_hi, mask_lo;
    unsigned int k_rem;         // rank (1-based) among the matching candidates
    unsigned int n_in;          // entries of the current candidate list
    unsigned int n_match;       // of them, how many match the decided prefix
    unsigned int cur;           // the current list: 0 = the dense list, 1, 2 = the scratch lists
};

struct TrimState {
    unsigned int size;          // live entries of the current table
    unsigned int k;             // entries to drop in this trim
    unsigned int invalid;       // malformed candidates seen by od_cache_insert
    unsigned int dropped;       // candidates that found no free slot on their whole probe sequence
    unsigned int n_live;        // entries of the dense list
    unsigned long long hi_and, hi_or;   // AND / OR of (new?, score) over the live entries: bits that never vary
    SelState sel[PASSES + 1];   // sel[p]: written by block 0 of pass p (sel[PASSES]: by the rebuild)
    unsigned int n_out[PASSES]; // entries pass p copied into its output list
    unsigned int hist[PASSES][256];
};

// Trim scratch for a table of `cap` slots: the dense list of live entries (order key and
// payload) and two lists of (hi, lo) candidates.
struct TrimLists {
    unsigned long long *r_hi, *r_key;
    int32_t *r_val;
    unsigned int *r_stamp, *r_freq, *r_born;
    unsigned long long *l_hi[2], *l_lo[2];
    unsigned int *grp_fill;             // [cap / OD_GROUP] slots handed out in each group of the table being built
};
__host__ __device__ inline TrimLists trim_lists(void *base, int64_t cap)
{
    TrimLists t;
    unsigned long long *q = (unsigned long long *)base;
    t.r_hi = q; t.r_key = q + cap;
    t.l_hi[0] = q + 2 * cap; t.l_lo[0] = q + 3 * cap;
    t.l_hi[1] = q + 4 * cap; t.l_lo[1] = q + 5 * cap;
    unsigned int *w = (unsigned int *)(q + 6 * cap);
    t.r_val = (int32_t *)w; t.r_stamp = w + cap; t.r_freq = w + 2 * cap; t.r_born = w + 3 * cap;
    t.grp_fill = w + 4 * cap;
    return t;
}
constexpr size_t TRIM_LIST_BYTES_PER_SLOT = 6 * 8 + 5 * 4;   // (the last array needs a 32nd of its share)

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

// The kernels of an insertion and of a trim form chains in which each needs what the one
// before it wrote. They are launched with programmatic stream serialization and wait at once:
// the launch latency of a kernel is spent while its predecessor still runs.
__device__ __forceinline__ void chain_wait()
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// launch with or without programmatic stream serialization (the context's "pdl" option)
template <typename... Params, typename... Args>
cudaError_t chain_launch(void (*kernel)(Params...), unsigned grid, unsigned block, cudaStream_t s, bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}


__global__ void insert_claim_kernel(int32_t N, int32_t v_q, int32_t v_p, const int32_t *__restrict__ runs,
                                    const int32_t *__restrict__ len, const int32_t *__restrict__ target,
                                    unsigned long long *keys, const int32_t *vals, int64_t cap,
                                    unsigned int *owner, int32_t *cand_slot, TrimState *st)
{
    chain_wait();
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
        // A group is filled from slot 0 without holes, and in a table at most half full it
        // rarely holds more than sixteen entries: its first sixteen keys are read at once
        // (one round trip instead of one per occupied slot), the rest one by one.
        constexpr int HEAD = 16;
        unsigned long long head[HEAD];
#pragma unroll
        for (int h = 0; h < HEAD / 2; ++h) {
            const ulonglong2 a = __ldcg((const ulonglong2 *)(keys + g * OD_GROUP) + h);
            head[2 * h] = a.x; head[2 * h + 1] = a.y;
        }
        int s0 = HEAD;                                      // the first slot that is empty or holds the key
#pragma unroll
        for (int h = HEAD - 1; h >= 0; --h)
            if (head[h] == 0ull || head[h] == key) s0 = h;
        for (int s = s0; s < OD_GROUP; ++s) {
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
    atomicAdd(&st->dropped, 1u);                            // the table is full: the candidate is lost
}

__global__ void insert_commit_kernel(int32_t N, const int32_t *__restrict__ target, int32_t *vals,
                                     unsigned int *stamp, unsigned int *freq, unsigned int *born,
                                     unsigned int *owner, const int32_t *__restrict__ cand_slot,
                                     unsigned int clock, TrimState *st)
{
    chain_wait();
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
    chain_wait();
    const unsigned int k = st->size > max_entries ? st->size - max_entries : 0u;
    if (threadIdx.x == 0) {
        st->k = k;
        st->n_live = 0u;
        st->hi_and = ~0ull; st->hi_or = 0ull;
        SelState z = {};
        z.k_rem = k;
        st->sel[0] = z;
    }
    for (int p = 0; p < PASSES; ++p) st->hist[p][threadIdx.x] = 0u;
    if (threadIdx.x < PASSES) st->n_out[threadIdx.x] = 0u;
}

// Exclusive offset of this thread's `n` items within the block's `total` (one block scan).
__device__ __forceinline__ unsigned int block_offsets(unsigned int n, unsigned int *s_warp, unsigned int &total)
{
    const unsigned int lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    unsigned int inc = n;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_up_sync(0xFFFFFFFFu, inc, off);
        if (lane >= off) inc += t;
    }
    __syncthreads();                                        // s_warp may still be read from the last call
    if (lane == 31u) s_warp[warp] = inc;
    __syncthreads();
    unsigned int base = 0;
    total = 0;
    for (unsigned int w = 0; w < blockDim.x / 32u; ++w) {
        if (w < warp) base += s_warp[w];
        total += s_warp[w];
    }
    return base + inc - n;
}

// One pass over the table: every live entry goes into the dense list (in no particular
// order: one append per block and iteration), and the spare table is cleared.
__global__ void trim_compact_kernel(int policy, unsigned int clock, const unsigned long long *keys,
                                    const int32_t *vals, const unsigned int *stamp, const unsigned int *freq,
                                    const unsigned int *born, unsigned long long *nkeys, int32_t *nvals,
                                    unsigned int *nstamp, unsigned int *nfreq, unsigned int *nborn,
                                    int64_t cap, void *lists, TrimState *st)
{
    __shared__ unsigned int s_warp[32];
    __shared__ unsigned int s_base;
    __shared__ unsigned long long s_and, s_or;
    chain_wait();
    const TrimLists L = trim_lists(lists, cap);
    if (threadIdx.x == 0) { s_and = ~0ull; s_or = 0ull; }
    unsigned long long t_and = ~0ull, t_or = 0ull;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x * 4;
    for (int64_t slot0 = (int64_t)blockIdx.x * blockDim.x * 4; slot0 < cap; slot0 += stride) {
        const int64_t slot = slot0 + (int64_t)threadIdx.x * 4;
        unsigned long long kk[4] = {0ull, 0ull, 0ull, 0ull};
        int vv[4] = {-1, -1, -1, -1};
        unsigned int ss[4] = {0, 0, 0, 0}, ff[4] = {0, 0, 0, 0}, bb[4] = {0, 0, 0, 0};
        if (slot < cap) {                                   // cap is a multiple of 64
            const ulonglong2 k01 = __ldg((const ulonglong2 *)(keys + slot));
            const ulonglong2 k23 = __ldg((const ulonglong2 *)(keys + slot) + 1);
            const int4 v4 = __ldg((const int4 *)(vals + slot));
            const uint4 s4 = __ldg((const uint4 *)(stamp + slot));
            const uint4 f4 = __ldg((const uint4 *)(freq + slot));
            const uint4 b4 = __ldg((const uint4 *)(born + slot));
            kk[0] = k01.x; kk[1] = k01.y; kk[2] = k23.x; kk[3] = k23.y;
            vv[0] = v4.x; vv[1] = v4.y; vv[2] = v4.z; vv[3] = v4.w;
            ss[0] = s4.x; ss[1] = s4.y; ss[2] = s4.z; ss[3] = s4.w;
            ff[0] = f4.x; ff[1] = f4.y; ff[2] = f4.z; ff[3] = f4.w;
            bb[0] = b4.x; bb[1] = b4.y; bb[2] = b4.z; bb[3] = b4.w;
            *(ulonglong2 *)(nkeys + slot) = make_ulonglong2(0ull, 0ull);
            *((ulonglong2 *)(nkeys + slot) + 1) = make_ulonglong2(0ull, 0ull);
            *(int4 *)(nvals + slot) = make_int4(-1, -1, -1, -1);
            *(uint4 *)(nstamp + slot) = make_uint4(0, 0, 0, 0);
            *(uint4 *)(nfreq + slot) = make_uint4(0, 0, 0, 0);
            *(uint4 *)(nborn + slot) = make_uint4(0, 0, 0, 0);
            if ((slot & (OD_GROUP - 1)) == 0) L.grp_fill[slot / OD_GROUP] = 0u;
        }
        unsigned int n = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) n += (kk[e] != 0ull && vv[e] >= 0) ? 1u : 0u;
        unsigned int total;
        unsigned int at = block_offsets(n, s_warp, total);
        if (threadIdx.x == 0) s_base = total ? atomicAdd(&st->n_live, total) : 0u;
        __syncthreads();
        at += s_base;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (kk[e] == 0ull || vv[e] < 0) continue;
            unsigned long long hi, lo;
            order_key(policy, clock, kk[e], ss[e], ff[e], bb[e], hi, lo);
            t_and &= hi; t_or |= hi;
            L.r_hi[at] = hi; L.r_key[at] = lo;
            L.r_val[at] = vv[e]; L.r_stamp[at] = ss[e]; L.r_freq[at] = ff[e]; L.r_born[at] = bb[e];
            ++at;
        }
    }
    // which bits of (new?, score) vary at all: AND and OR over the live entries
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        t_and &= __shfl_xor_sync(0xFFFFFFFFu, t_and, off);
        t_or |= __shfl_xor_sync(0xFFFFFFFFu, t_or, off);
    }
    if ((threadIdx.x & 31) == 0) { atomicAnd(&s_and, t_and); atomicOr(&s_or, t_or); }
    __syncthreads();
    if (threadIdx.x == 0) { atomicAnd(&st->hi_and, s_and); atomicOr(&st->hi_or, s_or); }
}

// Is digit `pass` the same in every live entry? Only asked for the five bytes of (new?, score).
__device__ __forceinline__ bool digit_is_constant(int pass, unsigned long long hi_and, unsigned long long hi_or)
{
    return pass < 5 && (((hi_or & ~hi_and) >> (8 * (4 - pass))) & 0xFFull) == 0ull;
}

// The state at the start of pass `pass` (0..PASSES), worked out from the state at the start of
// the pass before it and that pass's histogram: by every block alike, the same arithmetic on the
// same numbers. All threads of the block call; s_hist (256 words) and s_sel are its scratch.
__device__ __forceinline__ SelState select_state(int pass, const TrimState *st, unsigned int *s_hist, SelState *s_sel)
{
    if (pass == 0) {
        SelState z = st->sel[0];
        z.n_in = z.n_match = __ldcg(&st->n_live);
        return z;
    }
    const int q = pass - 1;                                  // the digit to settle
    s_hist[threadIdx.x] = __ldcg(&st->hist[q][threadIdx.x]);
    if (threadIdx.x == 0) {
        SelState t;
        const SelState *g = &st->sel[q];
        t.pre_hi = __ldcg(&g->pre_hi); t.pre_lo = __ldcg(&g->pre_lo);
        t.mask_hi = __ldcg(&g->mask_hi); t.mask_lo = __ldcg(&g->mask_lo);
        t.k_rem = __ldcg(&g->k_rem); t.n_in = __ldcg(&g->n_in);
        t.n_match = __ldcg(&g->n_match); t.cur = __ldcg(&g->cur);
        if (q == 0) t.n_in = t.n_match = __ldcg(&st->n_live);
        *s_sel = t;
    }
    const unsigned long long hi_and = __ldcg(&st->hi_and), hi_or = __ldcg(&st->hi_or);
    const unsigned int n_out = __ldcg(&st->n_out[q]);
    __syncthreads();
    if (threadIdx.x < 32) {
        SelState t = *s_sel;
        const int lane = threadIdx.x;
        unsigned int d, run = 0, in_bin = t.n_match;
        if (digit_is_constant(q, hi_and, hi_or)) {
            d = (unsigned int)(hi_or >> (8 * (4 - q))) & 0xFFu;   // every candidate has it: nothing else changes
        } else {
            // lane l owns bins 8l .. 8l+7; the first bin at which the running count reaches k_rem
            unsigned int mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) mine += s_hist[lane * 8 + i];
            unsigned int inc = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned int v = __shfl_up_sync(0xFFFFFFFFu, inc, off);
                if (lane >= off) inc += v;
            }
            const unsigned int reach = __ballot_sync(0xFFFFFFFFu, inc >= t.k_rem);
            const int owner = reach ? __ffs(reach) - 1 : 31;
            run = inc - mine; d = 255;
            if (lane == owner) {
                for (int i = 0; i < 8; ++i) {
                    if (run + s_hist[lane * 8 + i] >= t.k_rem) { d = lane * 8 + i; break; }
                    run += s_hist[lane * 8 + i];
                }
                if (d == 255u && !reach) run = inc;          // counts fell short: everything below the last bin
                in_bin = s_hist[d];
            }
            d = __shfl_sync(0xFFFFFFFFu, d, owner);
            run = __shfl_sync(0xFFFFFFFFu, run, owner);
            in_bin = __shfl_sync(0xFFFFFFFFu, in_bin, owner);
            // the pass copied its matching candidates if that at least halved a list worth copying
            if (2u * t.n_match <= t.n_in && t.n_in > 1024u) { t.cur = t.cur == 1u ? 2u : 1u; t.n_in = n_out; }
        }
        if (lane == 0) {
            t.k_rem -= run;
            t.n_match = in_bin;
            if (q < 5) {
                t.pre_hi |= (unsigned long long)d << (8 * (4 - q));
                t.mask_hi |= 0xFFull << (8 * (4 - q));
            } else {
                t.pre_lo |= (unsigned long long)d << (8 * (12 - q));
                t.mask_lo |= 0xFFull << (8 * (12 - q));
            }
            *s_sel = t;
        }
    }
    __syncthreads();
    return *s_sel;
}

// Pass `pass` of the radix select over the current candidate list: histogram of digit `pass`
// over the candidates that match the digits decided so far. If those are at most half of the
// list, they are copied into the other scratch list on the way (the next pass reads that one).
__global__ void trim_hist_kernel(int pass, int64_t cap, void *lists, TrimState *st)
{
    __shared__ unsigned int s_hist[256];
    __shared__ unsigned int s_warp[32];
    __shared__ unsigned int s_base;
    __shared__ SelState s_sel;
    chain_wait();
    if (st->k == 0u) return;                                 // nothing to drop: every block leaves
    const SelState S = select_state(pass, st, s_hist, &s_sel);
    if (blockIdx.x == 0 && threadIdx.x == 0) st->sel[pass] = S;
    if (digit_is_constant(pass, __ldcg(&st->hi_and), __ldcg(&st->hi_or))) return;   // the next pass fills it in
    __syncthreads();
    s_hist[threadIdx.x] = 0u;
    __syncthreads();
    const TrimLists L = trim_lists(lists, cap);
    const bool copy = 2u * S.n_match <= S.n_in && S.n_in > 1024u;   // short lists are not worth the copy
    const unsigned long long *in_hi = S.cur == 0u ? L.r_hi : L.l_hi[S.cur - 1u];
    const unsigned long long *in_lo = S.cur == 0u ? L.r_key : L.l_lo[S.cur - 1u];
    const unsigned int dst = S.cur == 1u ? 1u : 0u;          // scratch list 2 if list 1 is the input, else list 1
    unsigned long long *out_hi = L.l_hi[dst], *out_lo = L.l_lo[dst];
    // two entries per thread and iteration, both loads issued before the first use
    const unsigned int per_iter = gridDim.x * blockDim.x * 2u;
    for (unsigned int i0 = blockIdx.x * blockDim.x * 2u; i0 < S.n_in; i0 += per_iter) {
        const unsigned int i = i0 + threadIdx.x;
        const unsigned int j = i + blockDim.x;
        unsigned long long hi[2] = {0ull, 0ull}, lo[2] = {0ull, 0ull};
        bool ok[2] = {i < S.n_in, j < S.n_in};
        if (ok[0]) { hi[0] = __ldcg(in_hi + i); lo[0] = __ldcg(in_lo + i); }
        if (ok[1]) { hi[1] = __ldcg(in_hi + j); lo[1] = __ldcg(in_lo + j); }
        unsigned int n = 0;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            ok[e] = ok[e] && (hi[e] & S.mask_hi) == S.pre_hi && (lo[e] & S.mask_lo) == S.pre_lo;
            if (ok[e]) {
                // scores are heavily tied (most digits are equal across the table): one
                // shared-memory add per distinct digit of the warp, not one per entry
                const unsigned int d = digit_of(pass, hi[e], lo[e]);
                const unsigned int peers = __match_any_sync(__activemask(), d);
                if ((int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&s_hist[d], (unsigned int)__popc(peers));
                ++n;
            }
        }
        if (copy) {                                          // the same for every thread of the grid
            unsigned int total;
            unsigned int at = block_offsets(n, s_warp, total);
            if (threadIdx.x == 0) s_base = total ? atomicAdd(&st->n_out[pass], total) : 0u;
            __syncthreads();
            at += s_base;
#pragma unroll
            for (int e = 0; e < 2; ++e)
                if (ok[e]) { out_hi[at] = hi[e]; out_lo[at] = lo[e]; ++at; }
        }
    }
    __syncthreads();
    if (s_hist[threadIdx.x]) atomicAdd(&st->hist[pass][threadIdx.x], s_hist[threadIdx.x]);
}

// survivors of the dense list go into the (cleared) new table; which slot of its group an
// entry gets depends on timing, the set of entries does not
__global__ void trim_rebuild_kernel(unsigned long long *nkeys, int32_t *nvals, unsigned int *nstamp,
                                    unsigned int *nfreq, unsigned int *nborn, int64_t cap, void *lists,
                                    const TrimState *st)
{
    __shared__ unsigned int s_hist[256];
    __shared__ SelState s_sel;
    chain_wait();
    const TrimLists L = trim_lists(lists, cap);
    const unsigned int n = __ldcg(&st->n_live), k = st->k;
    unsigned long long thr_hi = 0ull, thr_lo = 0ull;
    if (k > 0u) {                                           // block-uniform
        const SelState S = select_state(PASSES, st, s_hist, &s_sel);
        thr_hi = S.pre_hi; thr_lo = S.pre_lo;
    }
    const uint64_t ngroups = (uint64_t)cap / OD_GROUP;
    for (unsigned int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const unsigned long long hi = L.r_hi[i], key = L.r_key[i];
        if (k > 0u && (hi < thr_hi || (hi == thr_hi && key <= thr_lo))) continue;   // among the k first: dropped
        const int32_t v = L.r_val[i];
        const unsigned int s = L.r_stamp[i], f = L.r_freq[i], b = L.r_born[i];
        uint64_t g = od_hash64(key) & (ngroups - 1);
        // A group is filled from its slot 0 without holes (od_cache_insert stops at the first
        // empty slot). Every placement takes the next slot of its group from the group's
        // counter: no two entries ever want the same slot, so there is nothing to retry and
        // a placement is one atomic add and five stores. A full group (32 entries: rare in a
        // table at most half full) sends the entry on to the next group, as a probe would go.
        for (uint64_t step = 0; step < ngroups; ++step) {
            const unsigned int at = atomicAdd(L.grp_fill + g, 1u);
            if (at < (unsigned int)OD_GROUP) {
                const int64_t ns = (int64_t)(g * OD_GROUP + at);
                nkeys[ns] = key; nvals[ns] = v; nstamp[ns] = s; nfreq[ns] = f; nborn[ns] = b;
                break;
            }
            g = (g + 1) & (ngroups - 1);
        }
    }
}

__global__ void trim_end_kernel(TrimState *st)
{
    chain_wait();
    st->size -= st->k; st->k = 0u;
}

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
                    c->d_born2, c->d_owner, c->d_cand_slot, c->d_trim, c->d_trim_lists};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    c->d_stamp = c->d_freq = c->d_born = c->d_stamp2 = c->d_freq2 = c->d_born2 = c->d_owner = nullptr;
    c->d_keys2 = nullptr; c->d_vals2 = nullptr; c->d_cand_slot = nullptr; c->d_trim = nullptr;
    c->d_trim_lists = nullptr;
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
    unsigned char *tl = nullptr;
    if (st == OD_OK) st = alloc_zero(&tl, (size_t)cap * TRIM_LIST_BYTES_PER_SLOT);
    c->d_trim_lists = tl;
    if (st != OD_OK) { od_cache_free_dynamic(c); return st; }
    OD_CUDA(cudaMemset(c->d_vals, 0xFF, (size_t)cap * sizeof(int32_t)));    // -1: no value
    OD_CUDA(cudaMemset(c->d_vals2, 0xFF, (size_t)cap * sizeof(int32_t)));
    OD_CUDA(cudaMemset(c->d_owner, 0xFF, (size_t)cap * sizeof(uint32_t)));
    c->cap = cap;
    c->table_written = true;
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
    c->table_written = true;
    const int threads = 128, blocks = (N + threads - 1) / threads;
    const bool pdl = c->opt_pdl != 0;
    OD_CUDA(chain_launch(insert_claim_kernel, (unsigned)blocks, (unsigned)threads, s, pdl, N, c->v_q, c->v_p, runs, len,
                         target, (unsigned long long *)c->d_keys, (const int32_t *)c->d_vals, c->cap,
                         c->d_owner, c->d_cand_slot, (TrimState *)c->d_trim));
    OD_CUDA(chain_launch(insert_commit_kernel, (unsigned)blocks, (unsigned)threads, s, pdl, N, target, c->d_vals,
                         c->d_stamp, c->d_freq, c->d_born, c->d_owner, (const int32_t *)c->d_cand_slot,
                         c->clock, (TrimState *)c->d_trim));
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
    c->table_written = true;
    TrimState *st = (TrimState *)c->d_trim;
    const int grid = c->sm_count * 4;
    const bool pdl = c->opt_pdl != 0;
    OD_CUDA(chain_launch(trim_begin_kernel, 1u, 256u, s, pdl, st, (unsigned int)c->dyn_max));
    OD_CUDA(chain_launch(trim_compact_kernel, (unsigned)grid, 256u, s, pdl, c->dyn_policy, c->clock,
                         (const unsigned long long *)c->d_keys, (const int32_t *)c->d_vals,
                         (const unsigned int *)c->d_stamp, (const unsigned int *)c->d_freq,
                         (const unsigned int *)c->d_born, (unsigned long long *)c->d_keys2, c->d_vals2,
                         c->d_stamp2, c->d_freq2, c->d_born2, c->cap, c->d_trim_lists, st));
    for (int pass = 0; pass < PASSES; ++pass)
        OD_CUDA(chain_launch(trim_hist_kernel, (unsigned)c->sm_count, 256u, s, pdl, pass, c->cap,
                             c->d_trim_lists, st));
    OD_CUDA(chain_launch(trim_rebuild_kernel, (unsigned)grid, 256u, s, pdl, (unsigned long long *)c->d_keys2,
                         c->d_vals2, c->d_stamp2, c->d_freq2, c->d_born2, c->cap, c->d_trim_lists,
                         (const TrimState *)st));
    OD_CUDA(chain_launch(trim_end_kernel, 1u, 1u, s, pdl, st));
    // the rebuilt table is the table for every call enqueued from now on
    std::swap(c->d_keys, c->d_keys2); std::swap(c->d_vals, c->d_vals2);
    std::swap(c->d_stamp, c->d_stamp2); std::swap(c->d_freq, c->d_freq2); std::swap(c->d_born, c->d_born2);
    return OD_OK;
}

int32_t od_cache_stats(od_ctx *c, int64_t *entries, int64_t *invalid, int64_t *dropped)
{
    if (!c) return OD_ERR_INVALID_ARG;
    if (!c->dyn) return OD_ERR_STATE;
    Guard g(c->device);
    if (!g.ok) return OD_ERR_CUDA;
    OD_CUDA(cudaDeviceSynchronize());
    unsigned int size = 0, inv = 0, drop = 0;
    const char *st = (const char *)c->d_trim;
    OD_CUDA(cudaMemcpy(&size, st + offsetof(TrimState, size), sizeof(size), cudaMemcpyDeviceToHost));
    OD_CUDA(cudaMemcpy(&inv, st + offsetof(TrimState, invalid), sizeof(inv), cudaMemcpyDeviceToHost));
    OD_CUDA(cudaMemcpy(&drop, st + offsetof(TrimState, dropped), sizeof(drop), cudaMemcpyDeviceToHost));
    if (entries) *entries = size;
    if (invalid) *invalid = inv;
    if (dropped) *dropped = drop;
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
