"""GPU parity of the online n-gram cache (insertion of unseen n-grams, LRU / LFU trim,
access stamping by od_map_proposals) against the dictionary oracle: table contents,
access clocks and frequencies are integers and must match exactly."""
import numpy as np
import pytest
import torch

from oracle import cache_policy as cp
from paper_2507_02659_b200 import binding as od

pytestmark = pytest.mark.gpu


def _universe(rng, n, v_q):
    lens = rng.integers(2, 5, size=n).astype(np.int32)
    runs = rng.integers(0, v_q, size=(n, 4)).astype(np.int32)
    return runs, lens


def _compare(ctx, ref):
    got = ctx.cache_dump()
    want = {k: (v[0], v[1], v[2]) for k, v in ref.entries.items()}
    assert len(got) == len(want)
    assert got == want


@pytest.mark.parametrize("policy", [cp.LRU, cp.LFU])
def test_insert_access_trim_match_the_oracle(cuda_device, policy):
    rng = np.random.default_rng(20 + policy)
    v_q, v_p, B, K = 60, 300, 16, 6
    vocab_map = np.where(rng.random(v_q) < 0.7, rng.permutation(v_p)[:v_q], -1).astype(np.int32)
    ctx = od.Context(cuda_device, v_q, v_p, B, K)
    ctx.set_vocab_map(vocab_map)
    ctx.cache_configure(40, policy, 64)
    ref = cp.DynamicCache(40, policy, v_q, v_p)
    uruns, ulens = _universe(rng, 120, v_q)
    utgt = rng.integers(0, v_p, size=120).astype(np.int32)
    dev = cuda_device
    for tick in range(1, 25):
        ctx.cache_set_clock(tick); ref.set_clock(tick)
        # a batch of proposals, most of them carrying a run of the universe
        d = rng.integers(0, v_q, size=(B, K)).astype(np.int32)
        klen = rng.integers(0, K + 1, size=B).astype(np.int32)
        for b in range(B):
            e = int(rng.integers(0, 120)); L = int(ulens[e])
            if L <= klen[b] and rng.random() < 0.8:
                o = int(rng.integers(0, klen[b] - L + 1)); d[b, o:o + L] = uruns[e, :L]
        q = rng.random((B, K)).astype(np.float32)
        mp = od.od_map_proposals(ctx, torch.from_numpy(d).to(dev), torch.from_numpy(klen).to(dev),
                                 torch.from_numpy(q).to(dev))
        torch.cuda.synchronize()
        for b in range(B):
            tgt, qp, ss, sl, m, stop = ref.map_sequence(vocab_map, d[b, :klen[b]], q[b])
            assert int(mp.m[b]) == m and bool(mp.tail_kind[b]) == stop
            assert mp.tgt_ids[b, :m].tolist() == tgt and mp.span_len[b, :m].tolist() == sl
            np.testing.assert_allclose(mp.q_prime[b, :m].cpu().numpy(), qp, rtol=1e-6)
        _compare(ctx, ref)
        # what "reverse translation" found this step: duplicates inside the batch (the
        # first wins), runs already cached, malformed candidates
        n = 20
        pick = rng.integers(0, 120, size=n)
        runs, lens, tg = uruns[pick].copy(), ulens[pick].copy(), utgt[pick].copy()
        tg[n // 2:] = rng.integers(0, v_p, size=n - n // 2)       # same run, another target: must lose
        lens[3] = 5; runs[5, 0] = v_q + 1; tg[7] = v_p              # malformed
        ctx.cache_insert(torch.from_numpy(runs).to(dev), torch.from_numpy(lens).to(dev),
                         torch.from_numpy(tg).to(dev))
        ref.insert_batch(runs, lens, tg)
        _compare(ctx, ref)
        if tick % 2 == 0:
            ctx.cache_trim(); ref.trim()
            assert len(ref) <= 40
            _compare(ctx, ref)
    ctx.close()


@pytest.mark.parametrize("policy", [cp.LRU, cp.LFU])
def test_large_batches_and_many_ties(cuda_device, policy):
    """Thousands of candidates per batch, most scores tied: the radix select has to
    resolve the order down to the run keys."""
    rng = np.random.default_rng(30 + policy)
    v_q, v_p = 32000, 128256
    ctx = od.Context(cuda_device, v_q, v_p, 4, 4)
    ctx.set_vocab_map(np.full(v_q, -1, np.int32))
    ctx.cache_configure(5000, policy, 4096)
    ref = cp.DynamicCache(5000, policy, v_q, v_p)
    uruns, ulens = _universe(rng, 20000, v_q)
    utgt = rng.integers(0, v_p, size=20000).astype(np.int32)
    dev = cuda_device
    evicted = 0
    for tick in range(1, 9):
        ctx.cache_set_clock(tick); ref.set_clock(tick)
        pick = np.where(rng.random(4096) < 0.5, (rng.zipf(1.3, size=4096) - 1) % 20000,
                        rng.integers(0, 20000, size=4096))
        runs, lens, tg = uruns[pick].copy(), ulens[pick].copy(), utgt[pick].copy()
        ctx.cache_insert(torch.from_numpy(runs).to(dev), torch.from_numpy(lens).to(dev),
                         torch.from_numpy(tg).to(dev))
        ref.insert_batch(runs, lens, tg)
        if tick % 3 == 0 or tick == 8:
            ctx.cache_trim(); evicted += ref.trim()
        _compare(ctx, ref)
    assert len(ref) == 5000 and evicted > 1000
    ctx.close()


def test_full_size_cache_fills_and_trims_to_its_bound(cuda_device):
    """262144 entries (the largest cache of the workloads): 20 batches of 16384 fresh
    candidates overfill it, the trim brings it back to exactly the bound."""
    rng = np.random.default_rng(40)
    v_q, v_p, cap = 32000, 128256, 262144
    ctx = od.Context(cuda_device, v_q, v_p, 4, 4)
    ctx.set_vocab_map(np.full(v_q, -1, np.int32))
    ctx.cache_configure(cap, cp.LRU, 16384)
    ref = cp.DynamicCache(cap, cp.LRU, v_q, v_p)
    dev = cuda_device
    for tick in range(1, 21):
        ctx.cache_set_clock(tick); ref.set_clock(tick)
        lens = rng.integers(2, 5, size=16384).astype(np.int32)
        runs = rng.integers(0, v_q, size=(16384, 4)).astype(np.int32)
        tg = rng.integers(0, v_p, size=16384).astype(np.int32)
        ctx.cache_insert(torch.from_numpy(runs).to(dev), torch.from_numpy(lens).to(dev),
                         torch.from_numpy(tg).to(dev))
        ref.insert_batch(runs, lens, tg)
    assert len(ref) > cap
    ctx.cache_trim(); ref.trim()
    assert len(ref) == cap
    _compare(ctx, ref)
    ctx.close()


def test_online_cache_argument_checks(cuda_device):
    ctx = od.Context(cuda_device, 100, 100, 4, 4)
    with pytest.raises(od.OdError) as e:
        ctx.cache_trim()                                  # no online cache yet
    assert e.value.status == -8
    with pytest.raises(od.OdError):
        ctx.cache_configure(10, 2, 8)                     # unknown policy
    ctx.cache_configure(10, cp.LFU, 8)
    z = torch.zeros(9, 4, dtype=torch.int32, device=cuda_device)
    with pytest.raises(od.OdError):                       # batch beyond max_insert
        ctx.cache_insert(z, torch.zeros(9, dtype=torch.int32, device=cuda_device),
                         torch.zeros(9, dtype=torch.int32, device=cuda_device))
    big = od.Context(cuda_device, 70000, 70000, 1, 2)
    with pytest.raises(od.OdError) as e:
        big.cache_configure(10, 0, 8)                     # ids do not fit 16 bits
    assert e.value.status == -5
    big.close(); ctx.close()


def test_translation_directly_behind_cache_writers_with_early_inputs(cuda_device):
    """With "early_inputs" the translation kernel reads the proposal before it waits for the launch
    in front of it, never the table. Nothing is synchronised between an insertion or a trim and
    the translations behind it: they must see the table those leave."""
    rng = np.random.default_rng(77)
    v_q, v_p, B, K = 60, 300, 32, 6
    vocab_map = np.where(rng.random(v_q) < 0.7, rng.permutation(v_p)[:v_q], -1).astype(np.int32)
    ctx = od.Context(cuda_device, v_q, v_p, B, K)
    ctx.set_vocab_map(vocab_map)
    ctx.cache_configure(40, cp.LRU, 64)
    ctx.set_option("early_inputs", 1)
    ref = cp.DynamicCache(40, cp.LRU, v_q, v_p)
    uruns, ulens = _universe(rng, 120, v_q)
    utgt = rng.integers(0, v_p, size=120).astype(np.int32)
    dev = cuda_device
    for tick in range(1, 13):
        ctx.cache_set_clock(tick); ref.set_clock(tick)
        props = []
        for _ in range(3):
            d = rng.integers(0, v_q, size=(B, K)).astype(np.int32)
            klen = rng.integers(0, K + 1, size=B).astype(np.int32)
            for b in range(B):
                e = int(rng.integers(0, 120)); L = int(ulens[e])
                if L <= klen[b] and rng.random() < 0.9:
                    o = int(rng.integers(0, klen[b] - L + 1)); d[b, o:o + L] = uruns[e, :L]
            q = rng.random((B, K)).astype(np.float32)
            props.append((d, klen, q, torch.from_numpy(d).to(dev), torch.from_numpy(klen).to(dev),
                          torch.from_numpy(q).to(dev)))
        pick = rng.integers(0, 120, size=30)
        runs, lens, tg = uruns[pick].copy(), ulens[pick].copy(), utgt[pick].copy()
        d_runs, d_lens, d_tg = (torch.from_numpy(x).to(dev) for x in (runs, lens, tg))
        torch.cuda.synchronize()                              # every input is resident from here on
        ctx.cache_insert(d_runs, d_lens, d_tg)
        mp0 = od.od_map_proposals(ctx, *props[0][3:])        # directly behind the insertion
        mp1 = od.od_map_proposals(ctx, *props[1][3:])        # behind another translation
        ctx.cache_trim()
        mp2 = od.od_map_proposals(ctx, *props[2][3:])        # directly behind the trim
        torch.cuda.synchronize()
        ref.insert_batch(runs, lens, tg)
        for i, mp in enumerate((mp0, mp1, mp2)):
            if i == 2:
                ref.trim()
            d, klen, q = props[i][:3]
            for b in range(B):
                tgt, qp, ss, sl, m, stop = ref.map_sequence(vocab_map, d[b, :klen[b]], q[b])
                assert int(mp.m[b]) == m and bool(mp.tail_kind[b]) == stop, (tick, i, b)
                assert mp.tgt_ids[b, :m].tolist() == tgt and mp.span_len[b, :m].tolist() == sl
        _compare(ctx, ref)
    ctx.close()


def test_a_full_table_counts_what_it_loses(cuda_device):
    """Insertions without a trim until the table (64 slots for a bound of 8 + 8) is full: every
    candidate is either in the cache or counted as lost, and malformed ones are counted too."""
    rng = np.random.default_rng(5)
    v_q, v_p = 200, 300
    ctx = od.Context(cuda_device, v_q, v_p, 4, 4)
    ctx.set_vocab_map(np.full(v_q, -1, np.int32))
    ctx.cache_configure(8, cp.LRU, 8)
    seen = set()
    bad = 0
    for tick in range(1, 16):
        ctx.cache_set_clock(tick)
        runs = np.full((8, 4), -1, np.int32); lens = np.full(8, 2, np.int32)
        for i in range(8):
            while True:
                r = tuple(int(x) for x in rng.integers(0, v_q, size=2))
                if r not in seen:
                    break
            seen.add(r); runs[i, :2] = r
        tg = rng.integers(0, v_p, size=8).astype(np.int32)
        if tick == 3:
            lens[0] = 7; seen.discard(tuple(int(x) for x in runs[0, :2])); bad += 1
        ctx.cache_insert(torch.from_numpy(runs).to(cuda_device), torch.from_numpy(lens).to(cuda_device),
                         torch.from_numpy(tg).to(cuda_device))
    entries, invalid, dropped = ctx.cache_stats()
    held = ctx.cache_dump()
    assert invalid == bad
    assert entries == len(held) == 64                 # every slot taken
    assert dropped == len(seen) - 64 and dropped > 0
    assert set(held) <= seen
    ctx.close()

