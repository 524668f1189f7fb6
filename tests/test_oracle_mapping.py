"""Pins for the oracle's translation step, Eq. (1) and Eq. (2) (CPU only)."""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _brute_force(d, vocab_map, cache_dict):
    """Every chain of consecutive valid pieces starting at offset 0 (a piece of
    length 1 needs a direct map, a longer piece must be a cached run); the
    greedy longest-first scan is the chain whose length vector is largest in
    lexicographic order (a chain that extends another one is larger)."""
    K = len(d)
    best = ()

    def rec(s, chain):
        nonlocal best
        if tuple(chain) > best:
            best = tuple(chain)
        if s == K:
            return
        for L in (1, 2, 3, 4):
            if s + L > K:
                continue
            if L == 1:
                ok = vocab_map[d[s]] >= 0
            else:
                ok = tuple(d[s:s + L]) in cache_dict
            if ok:
                rec(s + L, chain + [L])

    rec(0, [])
    return best


@pytest.mark.parametrize("seed", range(6))
def test_mapping_equals_brute_force_segmentation(seed):
    rng = np.random.default_rng(seed)
    V_q = 4
    vocab_map = np.array([10, 11, -1, 13], dtype=np.int32)
    if seed % 2:
        vocab_map = np.array([10, -1, -1, 13], dtype=np.int32)
    n_ent = int(rng.integers(1, 7))
    runs = np.full((n_ent, 4), -1, np.int32)
    lens = rng.integers(2, 5, size=n_ent).astype(np.int32)
    tg = (20 + np.arange(n_ent)).astype(np.int32)
    cache_dict = {}
    for e in range(n_ent):
        runs[e, :lens[e]] = rng.integers(0, V_q, size=lens[e])
        cache_dict.setdefault(tuple(int(x) for x in runs[e, :lens[e]]), int(tg[e]))
    cache = oracle.Cache(runs, lens, tg)
    assert len(cache) == len(cache_dict)
    for K in range(1, 7):
        for d in itertools.product(range(V_q), repeat=K):
            q = rng.random(K).astype(np.float32) * 0.9 + 0.05
            tgt, qp, ss, sl, m, tail, hits = oracle.map_sequence(cache, vocab_map, d, q)
            want = _brute_force(list(d), vocab_map, cache_dict)
            assert tuple(sl) == want, (d, tuple(sl), want)
            covered = int(sum(want))
            assert tail == (oracle.TAIL_UNMAPPED_STOP if covered < K else oracle.TAIL_COMPLETE)
            if tail == oracle.TAIL_UNMAPPED_STOP:
                assert ss[m] == covered
            s = 0
            for i, L in enumerate(want):
                assert ss[i] == s
                if L == 1:
                    assert tgt[i] == vocab_map[d[s]]
                    assert qp[i] == float(q[s])
                else:
                    assert tgt[i] == cache_dict[tuple(d[s:s + L])]
                    prod = 1.0
                    for j in range(L):
                        prod *= float(q[s + j])
                    assert qp[i] == pytest.approx(prod, rel=1e-15)
                s += L
            assert hits == sum(1 for L in want if L > 1)


def _patterns():
    out = []
    with open(os.path.join(GOLDEN, "merge_patterns.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, K, pieces, note = line.split()
            out.append((name, int(K), [int(x) for x in pieces.split(",")], note))
    return out


@pytest.mark.parametrize("name,K,pieces,note", _patterns())
def test_paper_merge_patterns(name, K, pieces, note):
    """Rebuild each pattern of the paper's examples with synthetic ids: the
    sub-tokens of a merged piece have no direct map unless the row is marked
    "direct", single pieces are directly mapped."""
    V_q = 64
    vocab_map = np.full(V_q, -1, np.int32)
    d, runs, lens, tg = [], [], [], []
    nxt = 1
    for i, L in enumerate(pieces):
        ids = list(range(nxt, nxt + L)); nxt += L
        d += ids
        if L == 1:
            vocab_map[ids[0]] = 100 + ids[0]
        else:
            if note == "direct":
                for x in ids:
                    vocab_map[x] = 100 + x
            runs.append(ids + [-1] * (4 - L)); lens.append(L); tg.append(500 + i)
    assert len(d) == K
    cache = oracle.Cache(np.array(runs, np.int32).reshape(-1, 4), np.array(lens, np.int32),
                         np.array(tg, np.int32))
    q = np.linspace(0.2, 0.8, K).astype(np.float32)
    tgt, qp, ss, sl, m, tail, hits = oracle.map_sequence(cache, vocab_map, d, q)
    assert list(sl) == pieces and m == len(pieces) and tail == oracle.TAIL_COMPLETE
    s = 0
    for i, L in enumerate(pieces):
        if L == 1:
            assert tgt[i] == 100 + d[s]
        else:
            assert tgt[i] == 500 + i
        assert qp[i] == pytest.approx(float(np.prod(q[s:s + L].astype(np.float64))), rel=1e-15)
        s += L


def test_run_cut_by_end_of_proposal_does_not_match():
    vocab_map = np.array([5, 6, 7, 8], np.int32)
    cache = oracle.Cache(np.array([[0, 1, 2, -1]], np.int32), np.array([3], np.int32),
                         np.array([9], np.int32))
    q = np.full(2, 0.5, np.float32)
    tgt, qp, ss, sl, m, tail, hits = oracle.map_sequence(cache, vocab_map, [0, 1], q)
    assert list(tgt) == [5, 6] and list(sl) == [1, 1] and hits == 0


def test_first_insertion_of_a_run_wins_and_lookup_matches_dict():
    rng = np.random.default_rng(3)
    E = 4000
    lens = rng.integers(2, 5, size=E).astype(np.int32)
    runs = np.full((E, 4), -1, np.int32)
    ref = {}
    tg = rng.integers(0, 1000, size=E).astype(np.int32)
    for e in range(E):
        runs[e, :lens[e]] = rng.integers(0, 6, size=lens[e])   # tiny alphabet: many repeats
        ref.setdefault(tuple(int(x) for x in runs[e, :lens[e]]), int(tg[e]))
    cache = oracle.Cache(runs, lens, tg)
    assert len(cache) == len(ref)
    for L in (2, 3, 4):
        for ids in itertools.product(range(7), repeat=L):
            assert cache.lookup(ids) == ref.get(tuple(ids), -1)


def test_malformed_entries_rejected():
    with pytest.raises(ValueError):
        oracle.Cache(np.array([[1, 2, 3, 4]], np.int32), np.array([5], np.int32),
                     np.array([1], np.int32))
    with pytest.raises(ValueError):
        oracle.Cache(np.array([[1, -1, -1, -1]], np.int32), np.array([1], np.int32),
                     np.array([1], np.int32))


def test_eq2_hand_example_and_mass_conservation():
    vals = {}
    with open(os.path.join(GOLDEN, "eq2_hand_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            vals[k] = np.array([float(x) for x in v])
    q_row = vals["q_row"].astype(np.float32)
    q2 = np.float32(vals["q_second"][0])
    vocab_map = np.arange(5, dtype=np.int32)
    prod = float(q_row[2]) * float(q2)
    qf = oracle.full_mapping(q_row, vocab_map, 6, first_draft_id=2, length=2,
                             ngram_token=5, ngram_prob=prod)
    np.testing.assert_allclose(qf, vals["q_full"], atol=1e-7)
    assert qf.sum() == pytest.approx(float(q_row.astype(np.float64).sum()), abs=1e-12)
    # a directly mapped position leaves the drafter's row untouched
    qd = oracle.full_mapping(q_row, vocab_map, 6, 2, 1, -1, 0.0)
    np.testing.assert_array_equal(qd[:5], q_row.astype(np.float64))
    assert qd[5] == 0.0
    # the prefix sub-token has no direct map: its left-over mass is dropped
    vm = vocab_map.copy(); vm[2] = -1
    qu = oracle.full_mapping(q_row, vm, 6, 2, 2, 5, prod)
    assert qu[2] == 0.0 and qu[5] == pytest.approx(prod)
    assert qu.sum() == pytest.approx(float(q_row.astype(np.float64).sum()) - float(q_row[2]) + prod)


def test_eq2_case_order_when_the_cases_collide():
    """Eq. (2) is piecewise: the n-gram's token takes the n-gram's probability even when it
    also has a direct pre-image, or when it is the image of the run's first sub-token."""
    vals = {}
    with open(os.path.join(GOLDEN, "eq2_hand_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            vals[k] = np.array([float(x) for x in v])
    q_row = vals["q_row"].astype(np.float32)
    prod = float(q_row[2]) * float(np.float32(vals["q_second"][0]))
    vocab_map = np.arange(5, dtype=np.int32)
    # (i) T = 3 has the direct pre-image 3
    qf = oracle.full_mapping(q_row, vocab_map, 6, first_draft_id=2, length=2, ngram_token=3, ngram_prob=prod)
    np.testing.assert_allclose(qf, vals["q_full_T_in_image"], atol=1e-7)
    # (ii) T = 2 = map[d_1]
    qf = oracle.full_mapping(q_row, vocab_map, 6, first_draft_id=2, length=2, ngram_token=2, ngram_prob=prod)
    np.testing.assert_allclose(qf, vals["q_full_T_is_prefix"], atol=1e-7)


def test_eq2_agrees_with_eq1_at_the_ngram_token_so_the_step_stays_lossless():
    """The acceptance test of a merged position uses q'(T) of Eq. (1); the residual of the same
    position uses q'(.) of Eq. (2). Speculative sampling returns p exactly only if both are the
    same number at T: min(p, q') + max(0, p - q') = p. Checked through the oracle's own
    translation (Eq. 1) and full mapping (Eq. 2) for targets outside the image, inside the
    image, and equal to the image of the first sub-token."""
    rng = np.random.default_rng(23)
    V_q, V_p = 12, 20
    vocab_map = np.full(V_q, -1, np.int32)
    md = rng.permutation(V_q)[:8]
    vocab_map[md] = rng.permutation(V_p)[:8]
    image = set(int(t) for t in vocab_map if t >= 0)
    outside = [t for t in range(V_p) if t not in image]
    seen = set()
    for trial in range(300):
        L = int(rng.integers(2, 5))
        run = rng.integers(0, V_q, size=L).astype(np.int32)
        d1 = int(run[0])
        kind = trial % 3
        if kind == 0:
            T = int(outside[rng.integers(0, len(outside))])
        elif kind == 1:
            T = int(vocab_map[md[rng.integers(0, len(md))]])
        else:
            if vocab_map[d1] < 0:
                continue
            T = int(vocab_map[d1])
        seen.add((kind, T in image, vocab_map[d1] == T))
        runs = np.full((1, 4), -1, np.int32); runs[0, :L] = run
        cache = oracle.Cache(runs, np.array([L], np.int32), np.array([T], np.int32))
        q_rows = rng.dirichlet(np.ones(V_q), size=L).astype(np.float32)
        q_sel = np.array([q_rows[j, run[j]] for j in range(L)], np.float32)
        tgt, qp, ss, sl, m, tail, hits = oracle.map_sequence(cache, vocab_map, run, q_sel)
        assert m == 1 and hits == 1 and tgt[0] == T and sl[0] == L
        qf = oracle.full_mapping(q_rows[0], vocab_map, V_p, d1, L, T, float(qp[0]))
        assert qf[T] == qp[0]
        p = rng.dirichlet(np.ones(V_p))
        # emitted mass at T: accepted proposal + residual draw after a rejection of T
        assert min(p[T], qp[0]) + max(0.0, p[T] - qf[T]) == pytest.approx(p[T], abs=1e-15)
        if vocab_map[d1] >= 0 and vocab_map[d1] != T:
            assert qf[vocab_map[d1]] == pytest.approx(float(q_rows[0, d1]) - qp[0], abs=1e-15)
    assert (1, True, False) in seen and any(k[2] for k in seen)


def test_full_mapping_through_a_random_partial_map():
    rng = np.random.default_rng(11)
    V_q, V_p = 50, 80
    q_row = rng.dirichlet(np.ones(V_q)).astype(np.float32)
    vocab_map = np.full(V_q, -1, np.int32)
    md = rng.permutation(V_q)[:35]
    vocab_map[md] = rng.permutation(V_p)[:35]
    qf = oracle.full_mapping(q_row, vocab_map, V_p, 0, 1, -1, 0.0)
    want = np.zeros(V_p)
    for d in range(V_q):
        if vocab_map[d] >= 0:
            want[vocab_map[d]] = float(q_row[d])
    np.testing.assert_array_equal(qf, want)
