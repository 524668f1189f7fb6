"""Pins of the online-cache oracle (Algorithm 1 cache update; App. D.5 eviction)."""
import collections

import numpy as np
import pytest

import oracle
from oracle import cache_policy as cp


def _cands(rng, n, v_q=50):
    lens = rng.integers(2, 5, size=n)
    runs = rng.integers(0, v_q, size=(n, 4))
    targets = rng.integers(0, 1000, size=n)
    return runs, lens, targets


def test_only_unseen_ngrams_are_added_and_the_first_wins():
    c = cp.DynamicCache(100, cp.LRU, 50, 1000)
    runs = np.array([[1, 2, 0, 0], [1, 2, 9, 9], [3, 4, 5, 0], [1, 2, 0, 0]])
    added = c.insert_batch(runs, [2, 2, 3, 2], [7, 8, 9, 10])
    assert added == 2 and c.lookup([1, 2]) == 7 and c.lookup([3, 4, 5]) == 9
    assert c.insert_batch(np.array([[1, 2, 0, 0]]), [2], [55]) == 0 and c.lookup([1, 2]) == 7
    # malformed candidates are skipped
    assert c.insert_batch(np.array([[1, 2, 3, 4], [60, 1, 0, 0], [1, 3, 0, 0]]), [5, 2, 2], [1, 1, 5000]) == 0


def test_trim_after_each_insertion_is_a_textbook_lru():
    """One item per tick, trim every tick, hits refresh recency: an OrderedDict LRU."""
    rng = np.random.default_rng(0)
    cap = 8
    c = cp.DynamicCache(cap, cp.LRU, 50, 1000)
    ref = collections.OrderedDict()
    universe = [tuple(int(x) for x in rng.integers(0, 50, size=2)) for _ in range(30)]
    for tick in range(1, 600):
        c.set_clock(tick)
        key = universe[int(rng.integers(0, len(universe)))]
        if c.lookup(key) >= 0:
            c.touch(key)
            ref.move_to_end(key)
        else:
            c.insert_batch(np.array([list(key) + [0, 0]]), [2], [tick % 1000])
            ref[key] = tick % 1000
            c.trim()
            while len(ref) > cap:
                ref.popitem(last=False)
        assert set(c.entries) == set(ref)
        assert all(c.entries[k][0] == ref[k] for k in ref)


def test_trim_after_each_insertion_is_a_brute_force_lfu():
    rng = np.random.default_rng(1)
    cap = 6
    c = cp.DynamicCache(cap, cp.LFU, 50, 1000)
    freq = {}
    universe = [tuple(int(x) for x in rng.integers(0, 50, size=3)) for _ in range(20)]
    weights = rng.random(len(universe)) ** 3
    weights /= weights.sum()
    for tick in range(1, 800):
        c.set_clock(tick)
        key = universe[int(rng.choice(len(universe), p=weights))]
        if key in freq:
            freq[key] += 1
            c.touch(key)
        else:
            if len(freq) == cap:                         # brute force: least frequent, ties by packed key
                victim = min(freq, key=lambda k: (freq[k], cp.packed_key(k)))
                del freq[victim]
            freq[key] = 1
            c.insert_batch(np.array([list(key) + [0]]), [3], [5])
            c.trim()
        assert {k: v[2] for k, v in c.entries.items()} == freq


@pytest.mark.parametrize("policy", [cp.LRU, cp.LFU])
def test_batched_trim_keeps_the_best_and_protects_the_current_tick(policy):
    rng = np.random.default_rng(2)
    c = cp.DynamicCache(40, policy, 50, 1000)
    for tick in range(1, 30):
        c.set_clock(tick)
        for key in list(c.entries)[:: max(1, int(rng.integers(1, 4)))]:
            c.touch(key)
        runs, lens, targets = _cands(rng, 12)
        c.insert_batch(runs, lens, targets)
        before = {k: list(v) for k, v in c.entries.items()}
        k = c.trim()
        assert len(c.entries) == min(len(before), 40) and k == len(before) - len(c.entries)
        gone = [before[x] for x in before if x not in c.entries]
        kept = [v for v in c.entries.values()]
        score = (lambda v: v[1]) if policy == cp.LRU else (lambda v: v[2])
        if gone:
            # nothing evicted is strictly better than something old that was kept
            old_kept = [score(v) for v in kept if v[3] != tick]
            if old_kept:
                assert max(score(v) for v in gone if v[3] != tick) <= min(old_kept) if any(v[3] != tick for v in gone) else True
            # entries learnt this tick go only when nothing older is left
            if any(v[3] == tick for v in gone):
                assert not old_kept


def test_tracked_translation_equals_the_static_one():
    """With the same contents the dictionary-based scan gives what the C oracle gives."""
    rng = np.random.default_rng(5)
    v_q, v_p = 40, 200
    vocab_map = np.where(rng.random(v_q) < 0.7, rng.permutation(v_p)[:v_q], -1).astype(np.int32)
    runs, lens, targets = _cands(rng, 60, v_q)
    targets = targets % v_p
    c = cp.DynamicCache(1000, cp.LRU, v_q, v_p)
    c.insert_batch(runs, lens, targets)
    static = oracle.Cache(runs, lens.astype(np.int32), targets.astype(np.int32))
    for _ in range(300):
        K = int(rng.integers(1, 9))
        d = rng.integers(0, v_q, size=K)
        if rng.random() < 0.7:                            # plant a cached run
            e = int(rng.integers(0, 60)); L = int(lens[e])
            if L <= K:
                o = int(rng.integers(0, K - L + 1)); d[o:o + L] = runs[e, :L]
        q = rng.random(K).astype(np.float32)
        tgt, qp, ss, sl, m, stop = c.map_sequence(vocab_map, d, q)
        t2, q2, s2, l2, m2, tail2, _ = oracle.map_sequence(static, vocab_map, d, q)
        assert m == m2 and stop == (tail2 == oracle.TAIL_UNMAPPED_STOP)
        assert tgt == list(t2) and sl == list(l2) and ss[:m] == list(s2)[:m]
        if stop:
            assert ss[m] == s2[m]
        np.testing.assert_allclose(qp, q2, rtol=1e-6)
