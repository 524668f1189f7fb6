"""Pins of the exit-rule oracle (Section 3.3, Eq. (4)-(6)) against what the
mathematics fixes: closed forms, monotonicity, a library product."""
import math

import numpy as np
import pytest

from oracle import exit_rule as er


def test_sigmoid_matches_the_definition_and_is_stable():
    for x in (-800.0, -30.0, -1.0, 0.0, 0.5, 30.0, 800.0):
        s = er.sigmoid(x)
        assert 0.0 <= s <= 1.0
        if abs(x) < 30:
            assert s == pytest.approx(1.0 / (1.0 + math.exp(-x)), rel=1e-15)
    assert er.sigmoid(0.0) == 0.5
    assert er.sigmoid(-800.0) == 0.0 and er.sigmoid(800.0) == 1.0


@pytest.mark.parametrize("x,gamma", [(2.0, 0.3), (2.0, 0.7), (0.3, 0.3), (4.0, 0.7), (-1.0, 0.5)])
def test_constant_head_gives_the_geometric_closed_form(x, gamma):
    """With sigma constant, 1 - sigma^k > gamma  <=>  k > log(1 - gamma)/log(sigma)."""
    K = 16
    s = 1.0 / (1.0 + math.exp(-x))
    k_closed = math.floor(math.log(1.0 - gamma) / math.log(s)) + 1
    length, reject = er.exit_rule(np.full((1, K), x), [K], gamma)
    assert int(length[0]) == min(k_closed, K)
    for k in range(K):
        assert reject[0, k] == pytest.approx(1.0 - s ** (k + 1), rel=1e-12, abs=1e-15)


def test_confident_head_never_exits_and_hopeless_head_exits_at_once():
    K = 10
    length, reject = er.exit_rule(np.full((2, K), 40.0), [K, 7], 0.3)
    assert list(length) == [K, 7] and reject.max() < 1e-15
    length, _ = er.exit_rule(np.full((1, K), -40.0), [K], 0.99)
    assert int(length[0]) == 1
    length, _ = er.exit_rule(np.full((1, K), 0.0), [0], 0.3)
    assert int(length[0]) == 0


def test_product_against_the_library_and_strict_inequality():
    rng = np.random.default_rng(3)
    f = rng.normal(1.5, 1.5, size=(50, 8))
    length, reject = er.exit_rule(f, np.full(50, 8), 0.5)
    for b in range(50):
        sig = [1.0 / (1.0 + math.exp(-v)) for v in f[b]]
        for k in range(8):
            assert reject[b, k] == pytest.approx(1.0 - math.prod(sig[:k + 1]), rel=1e-13, abs=1e-15)
        over = [k + 1 for k in range(8) if 1.0 - math.prod(sig[:k + 1]) > 0.5]
        assert int(length[b]) == (over[0] if over else 8)
    # exactly gamma does not fire: sigma = 1/2, gamma = 1/2 -> fires at k = 2 (3/4 > 1/2), not at k = 1
    length, reject = er.exit_rule(np.zeros((1, 4)), [4], 0.5)
    assert reject[0, 0] == 0.5 and int(length[0]) == 2


def test_monotone_in_gamma_and_in_the_head_outputs():
    rng = np.random.default_rng(4)
    f = rng.normal(1.0, 2.0, size=(200, 12))
    avail = rng.integers(0, 13, size=200)
    prev = None
    for gamma in (0.1, 0.3, 0.5, 0.7, 0.9):
        length, _ = er.exit_rule(f, avail, gamma)
        assert (length <= avail).all()
        if prev is not None:
            assert (length >= prev).all()        # a laxer threshold never shortens the draft
        prev = length
    base, _ = er.exit_rule(f, avail, 0.5)
    more, _ = er.exit_rule(f + 0.7, avail, 0.5)  # a more confident head never shortens it either
    assert (more >= base).all()
