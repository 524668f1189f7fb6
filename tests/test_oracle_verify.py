"""Pins for the oracle's softmax / acceptance / residual / free-token steps
(Algorithm 1, verification lines; residual of the notation paragraph)."""
import numpy as np
import pytest
import scipy.special
import torch

import oracle


def _run(vocab_map, v_p, draft_ids, q_rows, logits, T=1.0, seeds=None, step=0,
         cache=None, draft_len=None, probe=None):
    draft_ids = np.asarray(draft_ids, np.int32)
    B, K = draft_ids.shape
    if cache is None:
        cache = oracle.Cache(np.zeros((0, 4), np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32))
    if seeds is None:
        seeds = np.arange(B, dtype=np.uint64)
    if draft_len is None:
        draft_len = np.full(B, K, np.int32)
    q_rows = np.asarray(q_rows, np.float32)
    q_sel = np.take_along_axis(q_rows, draft_ids[..., None].astype(np.int64), axis=2)[..., 0]
    temps = np.full(B, T, np.float32) if np.isscalar(T) else np.asarray(T, np.float32)
    return oracle.step_batch(cache, vocab_map, v_p, draft_ids, draft_len, q_sel, q_rows,
                             np.asarray(logits, np.float32), oracle.DTYPE_F32, temps, seeds,
                             step, probe_token=probe)


def _first_emitted(res, pos=0):
    """Token the step emits at position `pos` (accepted proposal or the extra
    token), or -1 where the step ended before `pos`."""
    n = res.n_accepted
    out = np.full(n.shape[0], -1, np.int64)
    acc = n > pos
    out[acc] = res.tgt_ids[acc, pos]
    ext = n == pos
    out[ext] = res.token[ext]
    return out


def _chi2_ok(counts, p, sigmas=5.0):
    n = counts.sum()
    e = n * p
    keep = e > 0
    chi2 = ((counts[keep] - e[keep]) ** 2 / e[keep]).sum()
    dof = keep.sum() - 1
    return chi2 < dof + sigmas * np.sqrt(2 * dof), chi2


def _softmax64(x, T):
    return scipy.special.softmax(np.asarray(x, np.float64) / T, axis=-1)


# ---------------------------------------------------------------- softmax
@pytest.mark.parametrize("T", [1.0, 0.7, 0.01])
def test_softmax_row_equals_library_softmax(T):
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(1000) * 3).astype(np.float32)
    p = oracle.softmax_row(x, T)
    np.testing.assert_allclose(p, _softmax64(x, T), rtol=1e-12, atol=1e-300)
    pt = torch.softmax(torch.from_numpy(x).double() / T, dim=0).numpy()
    np.testing.assert_allclose(p, pt, rtol=1e-12, atol=1e-300)
    assert p.sum() == pytest.approx(1.0, abs=1e-12)


def test_softmax_row_decodes_bf16_exactly():
    rng = np.random.default_rng(1)
    xb = torch.from_numpy((rng.standard_normal(777) * 3).astype(np.float32)).bfloat16()
    bits, code = oracle.logits_to_numpy(xb)
    assert code == oracle.DTYPE_BF16
    p = oracle.softmax_row(bits, 0.5)
    np.testing.assert_allclose(p, _softmax64(xb.float().numpy(), 0.5), rtol=1e-12)


def test_row_stats_reported_by_step():
    rng = np.random.default_rng(2)
    V, K = 97, 3
    logits = (rng.standard_normal((2, K + 1, V)) * 3).astype(np.float32)
    q_rows = rng.dirichlet(np.ones(V), size=(2, K)).astype(np.float32)
    d = rng.integers(0, V, size=(2, K))
    res = _run(np.arange(V, dtype=np.int32), V, d, q_rows, logits, T=0.7)
    for b in range(2):
        for r in range(K + 1):
            x = logits[b, r].astype(np.float64)
            assert res.row_max[b, r] == x.max()
            assert res.row_sum[b, r] == pytest.approx(np.exp((x - x.max()) / np.float64(np.float32(0.7))).sum(), rel=1e-12)
        for i in range(K):
            assert res.p_sel[b, i] == pytest.approx(_softmax64(logits[b, i], np.float64(np.float32(0.7)))[d[b, i]], rel=1e-11)


# ------------------------------------------------- lossless invariant (P1)
def _mc_problem(rng, V_q, V_p, K, n, vocab_map, T=1.0):
    zq = rng.standard_normal((K, V_q)) * 1.5
    zq[:, vocab_map < 0] += 2.0          # unmapped ids carry real mass
    zp = rng.standard_normal((K + 1, V_p)) * 1.5
    q = _softmax64(zq, 1.0).astype(np.float32)
    q64 = q.astype(np.float64)
    q64 /= q64.sum(axis=1, keepdims=True)
    d = np.stack([rng.choice(V_q, size=n, p=q64[j]) for j in range(K)], axis=1)
    q_rows = np.broadcast_to(q, (n, K, V_q))
    logits = np.broadcast_to(zp.astype(np.float32), (n, K + 1, V_p))
    return d, q_rows, logits, zp.astype(np.float32), q


@pytest.mark.parametrize("K", [1, 4])
@pytest.mark.parametrize("unmapped", [0, 3])
def test_lossless_first_and_second_token_distribution(K, unmapped):
    """Speculative sampling is lossless: with proposals drawn from q, every
    emitted token is distributed as the target p, also when some draft ids have
    no direct map and stop the proposal (forced rejection + residual)."""
    rng = np.random.default_rng(100 + K + unmapped)
    V = 8
    vocab_map = np.arange(V, dtype=np.int32)
    if unmapped:
        vocab_map = np.array([3, -1, 0, 7, -1, 5, -1, 2], dtype=np.int32)
    n = 400_000
    d, q_rows, logits, zp, q = _mc_problem(rng, V, V, K, n, vocab_map)
    res = _run(vocab_map, V, d, q_rows, logits, seeds=np.arange(n, dtype=np.uint64) + 12345, step=9)
    p0 = _softmax64(zp[0], 1.0)
    t0 = _first_emitted(res, 0)
    assert (t0 >= 0).all()
    c0 = np.bincount(t0, minlength=V).astype(np.float64)
    ok, chi2 = _chi2_ok(c0, p0)
    assert ok, chi2
    assert np.abs(c0 / n - p0).max() < 5 * np.sqrt(0.25 / n)
    if K > 1:
        t1 = _first_emitted(res, 1)
        sel = t1 >= 0
        assert sel.sum() > n // 20
        c1 = np.bincount(t1[sel], minlength=V).astype(np.float64)
        ok, chi2 = _chi2_ok(c1, _softmax64(zp[1], 1.0))
        assert ok, chi2
    if unmapped:
        # the test has teeth: sampling the extra token from p (instead of the
        # residual) after an unmapped stop at position 0 gives a different law
        stop0 = (res.m == 0)
        assert stop0.sum() > n // 50
        wrong = t0.copy()
        u = res.u_samp[stop0]
        wrong[stop0] = np.searchsorted(np.cumsum(p0), u, side="right").clip(0, V - 1)
        cw = np.bincount(wrong, minlength=V).astype(np.float64)
        ok_wrong, _ = _chi2_ok(cw, p0)
        assert not ok_wrong


def test_acceptance_probability_closed_form():
    """P(accept at one position) = sum_t min(p(t), q'(t)); with identical rows
    the accepted length is geometric: E[n] = sum_{i=1..K} alpha^i."""
    rng = np.random.default_rng(7)
    V, K, n = 8, 4, 400_000
    zq = rng.standard_normal(V) * 1.5
    zp = rng.standard_normal(V) * 1.5
    q = _softmax64(zq, 1.0).astype(np.float32)
    q64 = q.astype(np.float64) / q.astype(np.float64).sum()
    d = rng.choice(V, size=(n, K), p=q64)
    q_rows = np.broadcast_to(q, (n, K, V))
    logits = np.broadcast_to(zp.astype(np.float32), (n, K + 1, V))
    res = _run(np.arange(V, dtype=np.int32), V, d, q_rows, logits,
               seeds=np.arange(n, dtype=np.uint64) * 3 + 1, step=4)
    p = _softmax64(zp.astype(np.float32), 1.0)
    alpha = np.minimum(p, q.astype(np.float64)).sum()
    first = res.accept[:, 0].mean()
    assert abs(first - alpha) < 5 * np.sqrt(alpha * (1 - alpha) / n)
    want_len = sum(alpha ** i for i in range(1, K + 1))
    assert abs(res.n_accepted.mean() - want_len) < 5 * np.sqrt(K * K / n)
    # prefix rule: n = number of leading accepts
    lead = np.cumprod(res.accept, axis=1).sum(axis=1)
    np.testing.assert_array_equal(lead, res.n_accepted)
    # residual mass at a rejection = 1 - alpha
    rej = res.kind == oracle.KIND_RESIDUAL
    np.testing.assert_allclose(res.mass[rej], 1 - alpha, rtol=1e-6)
    np.testing.assert_allclose(res.mass[~rej], 1.0, rtol=1e-12)


# ------------------------------------------------------ special cases (P5)
def test_identical_distributions_accept_everything_then_bonus():
    rng = np.random.default_rng(8)
    V, K, n = 16, 5, 2000
    z = (rng.standard_normal((n, K + 1, V)) * 2).astype(np.float32)
    q_rows = _softmax64(z[:, :K], 1.0).astype(np.float32)
    d = rng.integers(0, V, size=(n, K))
    res = _run(np.arange(V, dtype=np.int32), V, d, q_rows, z)
    # p == q up to fp32 rounding of q: ratio is 1 or within 1e-6 of it
    assert (res.ratio[:, :K] > 1 - 1e-6).all()
    full = res.n_accepted == K
    assert full.mean() > 0.999
    assert (res.kind[full] == oracle.KIND_BONUS).all()
    # free token: plain categorical inverse-CDF draw from p_m
    for b in np.nonzero(full)[0][:200]:
        p = _softmax64(z[b, K], 1.0)
        c = np.cumsum(p)
        want = int(np.searchsorted(c, res.u_samp[b] * c[-1], side="right"))
        assert res.token[b] == min(want, V - 1)
        assert res.u_samp[b] == oracle.uniform(int(b), 0, K, 1)


def test_low_temperature_accepts_exactly_the_argmax():
    rng = np.random.default_rng(9)
    V, K, n = 32, 3, 3000
    z = (rng.standard_normal((n, K + 1, V)) * 3).astype(np.float32)
    # keep the top-2 gap away from zero so T = 0.01 separates them fully
    srt = np.sort(z, axis=-1)
    z[(srt[..., -1] - srt[..., -2]) < 0.5] += 0  # no-op; gaps filtered below
    q_rows = np.full((n, K, V), 1.0 / V, np.float32)
    d = rng.integers(0, V, size=(n, K))
    for b in range(0, n, 2):           # make half of the proposals the argmax
        d[b] = z[b, :K].argmax(-1)
    res = _run(np.arange(V, dtype=np.int32), V, d, q_rows, z, T=0.01)
    gap_ok = (srt[..., -1] - srt[..., -2])[:, :K] > 0.5
    is_max = d == z[:, :K].argmax(-1)
    sure = gap_ok
    assert (res.accept[sure & is_max] == 1).all()
    # a non-argmax token has p ~ exp(-50) or less: rejected unless u is tiny
    assert res.accept[sure & ~is_max].mean() < 1e-3
    # the extra token after a rejection is the argmax (residual mass sits there)
    rej = (res.n_accepted < K)
    rows = res.n_accepted[rej]
    bs = np.nonzero(rej)[0]
    good = gap_ok[bs, rows]
    assert (res.token[bs][good] == z[bs, rows].argmax(-1)[good]).all()


def test_bonus_only_when_everything_is_accepted_and_draft_count():
    rng = np.random.default_rng(10)
    V_q, V_p, K, n = 12, 20, 6, 4000
    vocab_map = np.full(V_q, -1, np.int32)
    vocab_map[:9] = rng.permutation(V_p)[:9]
    runs = np.array([[9, 10, -1, -1], [10, 11, 9, -1]], np.int32)
    cache = oracle.Cache(runs, np.array([2, 3], np.int32), np.array([18, 19], np.int32))
    assert 18 not in vocab_map and 19 not in vocab_map
    q_rows = rng.dirichlet(np.ones(V_q), size=(n, K)).astype(np.float32)
    logits = (rng.standard_normal((n, K + 1, V_p)) * 2).astype(np.float32)
    d = rng.integers(0, V_q, size=(n, K))
    klen = rng.integers(1, K + 1, size=n).astype(np.int32)
    res = _run(vocab_map, V_p, d, q_rows, logits, cache=cache, draft_len=klen)
    assert (res.hits > 0).sum() > 50
    assert (res.tail_kind == oracle.TAIL_UNMAPPED_STOP).sum() > 50
    for b in range(n):
        m, nacc = res.m[b], res.n_accepted[b]
        assert 0 <= nacc <= m <= klen[b]
        bonus = res.kind[b] == oracle.KIND_BONUS
        assert bonus == (nacc == m and res.tail_kind[b] == oracle.TAIL_COMPLETE)
        assert res.n_draft_accepted[b] == res.span_len[b, :nacc].sum()
        if res.tail_kind[b] == oracle.TAIL_COMPLETE:
            assert res.span_len[b, :m].sum() == klen[b]
        assert 0 <= res.token[b] < V_p
        assert res.cdf_lo[b] <= res.u_samp[b] * res.mass[b] < res.cdf_hi[b] or \
            res.cdf_hi[b] == pytest.approx(res.mass[b])


def test_residual_uses_eq2_at_a_rejected_ngram():
    """At a rejected n-gram position the residual is max(0, p - q') with q' of
    Eq. (2); checked against numpy on the oracle's own Eq. (2) vector (itself
    pinned by the hand example)."""
    rng = np.random.default_rng(12)
    V_q, V_p, K = 6, 9, 3
    vocab_map = np.array([0, 1, 2, 3, 4, 5], np.int32)
    cache = oracle.Cache(np.array([[2, 4, -1, -1]], np.int32), np.array([2], np.int32),
                         np.array([7], np.int32))
    n = 5000
    q_rows = rng.dirichlet(np.ones(V_q) * 3, size=(n, K)).astype(np.float32)
    logits = (rng.standard_normal((n, K + 1, V_p))).astype(np.float32)
    logits[:, 0, 7] -= 6.0           # the n-gram token is unlikely under p: often rejected
    d = np.tile(np.array([2, 4, 1]), (n, 1))
    res = _run(vocab_map, V_p, d, q_rows, logits, cache=cache)
    assert (res.m == 2).all() and (res.span_len[:, 0] == 2).all() and (res.tgt_ids[:, 0] == 7).all()
    rej0 = np.nonzero(res.n_accepted == 0)[0]
    assert rej0.size > 500
    for b in rej0[:300]:
        p = _softmax64(logits[b, 0], 1.0)
        prod = float(q_rows[b, 0, 2]) * float(q_rows[b, 1, 4])
        qf = oracle.full_mapping(q_rows[b, 0], vocab_map, V_p, 2, 2, 7, prod)
        r = np.maximum(0.0, p - qf)
        c = np.cumsum(r)
        assert res.mass[b] == pytest.approx(c[-1], rel=1e-12)
        want = int(np.searchsorted(c, res.u_samp[b] * c[-1], side="right"))
        assert res.token[b] == want
        assert res.u_samp[b] == oracle.uniform(int(b), 0, 0, 1)


def test_zero_residual_mass_falls_back_to_target_distribution():
    V, K = 6, 1
    z = np.zeros((1, K + 1, V), np.float32)
    # q' >= p everywhere except nowhere: q = p exactly representable (uniform 1/6 is
    # not, so use V = 8)
    V = 8
    z = np.zeros((1, K + 1, V), np.float32)
    q_rows = np.full((1, K, V), 0.125, np.float32)
    # force a rejection with an unmapped proposal: q' covers all mapped ids, p == q'
    vocab_map = np.arange(V, dtype=np.int32)
    res = None
    for seed in range(64):
        r = _run(vocab_map, V, [[3]], q_rows, z, seeds=np.array([seed], np.uint64))
        assert r.ratio[0, 0] == 1.0 and r.n_accepted[0] == 1
    # make position 0 an unmapped stop with p <= q' on the image and no mass outside it
    vm = np.array([0, 1, 2, 3, 4, 5, 6, -1], np.int32)
    z2 = np.zeros((1, 2, 7), np.float32)
    q2 = np.zeros((1, 1, 8), np.float32)
    q2[0, 0, :7] = 0.142857148      # >= 1/7 in fp32
    q2[0, 0, 7] = 0.0
    r = _run(vm, 7, [[7]], q2, z2)
    assert r.m[0] == 0 and r.tail_kind[0] == oracle.TAIL_UNMAPPED_STOP
    assert r.flags[0] & oracle.FLAG_ZERO_MASS
    assert 0 <= r.token[0] < 7
    assert r.mass[0] == pytest.approx(1.0)


def test_bad_temperature_is_flagged():
    V, K = 8, 2
    z = np.zeros((1, K + 1, V), np.float32)
    q_rows = np.full((1, K, V), 0.125, np.float32)
    r = _run(np.arange(V, dtype=np.int32), V, [[1, 2]], q_rows, z, T=0.0)
    assert r.flags[0] & oracle.FLAG_BAD_TEMPERATURE
    assert r.token[0] == -1


def test_threads_do_not_change_results():
    rng = np.random.default_rng(13)
    V, K, n = 50, 4, 64
    q_rows = rng.dirichlet(np.ones(V), size=(n, K)).astype(np.float32)
    logits = (rng.standard_normal((n, K + 1, V)) * 2).astype(np.float32)
    d = rng.integers(0, V, size=(n, K)).astype(np.int32)
    cache = oracle.Cache(np.zeros((0, 4), np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32))
    q_sel = np.take_along_axis(q_rows, d[..., None].astype(np.int64), axis=2)[..., 0]
    args = (cache, np.arange(V, dtype=np.int32), V, d, np.full(n, K, np.int32), q_sel, q_rows,
            logits, oracle.DTYPE_F32, np.ones(n, np.float32), np.arange(n, dtype=np.uint64), 3)
    a = oracle.step_batch(*args, threads=1)
    b = oracle.step_batch(*args, threads=4)
    for f in ("tgt_ids", "n_accepted", "token", "p_sel", "mass", "row_sum"):
        np.testing.assert_array_equal(getattr(a, f), getattr(b, f))
