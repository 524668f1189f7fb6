"""Pins of the distillation-loss oracle (Section 3.2, Eq. (3))."""
import numpy as np
import pytest
import torch

from oracle import distill as ds


def _softmax(z):
    z = np.asarray(z, np.float64)
    e = np.exp(z - z.max())
    return e / e.sum()


def test_kl_and_gradient_against_torch_on_an_identity_map():
    """Identity map, full support: KL(q || p) and its gradient through softmax are
    what torch's kl_div and autograd give."""
    rng = np.random.default_rng(0)
    V = 50
    z = torch.tensor(rng.normal(0, 2, V), dtype=torch.float64, requires_grad=True)
    x = rng.normal(0, 2, V)
    T = 0.7
    log_p = torch.log_softmax(torch.tensor(x) / T, dim=0)
    log_q = torch.log_softmax(z, dim=0)
    ref = torch.nn.functional.kl_div(log_p, log_q, reduction="sum", log_target=True)   # KL(q || p)
    ref.backward()
    loss, grad = ds.position_kl(_softmax(z.detach().numpy()), ds.log_softmax_row(x, T), np.arange(V))
    assert loss == pytest.approx(float(ref), rel=1e-12)
    np.testing.assert_allclose(grad, z.grad.numpy(), rtol=1e-10, atol=1e-14)


@pytest.mark.parametrize("seed", range(3))
def test_gradients_against_central_differences_with_a_partial_map(seed):
    rng = np.random.default_rng(seed)
    V_q, V_p = 12, 30
    vocab_map = np.where(rng.random(V_q) < 0.7, rng.permutation(V_p)[:V_q], -1)
    z = rng.normal(0, 1.5, V_q)
    log_p = ds.log_softmax_row(rng.normal(0, 2, V_p), 1.0)
    f_kl = lambda zz: ds.position_kl(_softmax(zz), log_p, vocab_map)[0]
    f_nll = lambda zz: ds.position_nll(_softmax(zz), 3, 0.2)[0]
    _, g_kl = ds.position_kl(_softmax(z), log_p, vocab_map)
    _, g_nll = ds.position_nll(_softmax(z), 3, 0.2)
    h = 1e-6
    for d in range(V_q):
        e = np.zeros(V_q); e[d] = h
        assert g_kl[d] == pytest.approx((f_kl(z + e) - f_kl(z - e)) / (2 * h), abs=2e-8)
        assert g_nll[d] == pytest.approx((f_nll(z + e) - f_nll(z - e)) / (2 * h), abs=2e-8)


def test_kl_is_nonnegative_and_zero_only_when_equal_on_a_full_map():
    rng = np.random.default_rng(1)
    V = 20
    ident = np.arange(V)
    for _ in range(50):
        q = _softmax(rng.normal(0, 2, V))
        x = rng.normal(0, 2, V)
        loss, _ = ds.position_kl(q, ds.log_softmax_row(x, 1.0), ident)
        assert loss > 0
    x = rng.normal(0, 2, V)
    loss, grad = ds.position_kl(_softmax(x), ds.log_softmax_row(x, 1.0), ident)
    assert abs(loss) < 1e-14 and np.abs(grad).max() < 1e-14


def test_gradient_identities():
    rng = np.random.default_rng(2)
    V_q, V_p = 40, 90
    vocab_map = np.where(rng.random(V_q) < 0.6, rng.permutation(V_p)[:V_q], -1)
    q = _softmax(rng.normal(0, 2, V_q))
    log_p = ds.log_softmax_row(rng.normal(0, 2, V_p), 0.5)
    loss, grad = ds.position_kl(q, log_p, vocab_map)
    assert abs(grad.sum()) < 1e-14                       # gradients through a softmax sum to zero
    mass = q[vocab_map >= 0].sum()
    # sum_d q(d) g(d) = loss + mapped mass, so an unmapped id gets -q(d) * (loss + mass)
    unm = np.nonzero(vocab_map < 0)[0]
    np.testing.assert_allclose(grad[unm], -q[unm] * (loss + mass), rtol=1e-12)
    l2, g2 = ds.position_nll(q, 7, 0.2)
    assert l2 == pytest.approx(-0.2 * np.log(q[7])) and abs(g2.sum()) < 1e-15 and g2[7] == pytest.approx(0.2 * (q[7] - 1))


def test_sequence_masks_follow_the_pieces():
    """Pieces (1, 3, 1) of a 5-token proposal (the overview figure's pattern): KL at the
    single tokens, NLL at the three sub-tokens; nothing after an unmapped stop."""
    rng = np.random.default_rng(3)
    V_q, V_p, K = 10, 25, 6
    vocab_map = np.arange(V_q)
    q_rows = np.stack([_softmax(rng.normal(0, 1, V_q)) for _ in range(K)])
    logits = rng.normal(0, 2, (K + 1, V_p))
    d = rng.integers(0, V_q, K)
    loss, grad = ds.distill_sequence(q_rows, d, [0, 1, 4], [1, 3, 1], 3, logits, 1.0, vocab_map, [d[0], 20, d[4]], 0.2)
    assert loss[5] == 0 and not grad[5].any()
    for j in (1, 2, 3):
        assert loss[j] == pytest.approx(-0.2 * np.log(q_rows[j, d[j]]))
    l0, _ = ds.position_kl(q_rows[0], ds.log_softmax_row(logits[0], 1.0), vocab_map)
    l4, _ = ds.position_kl(q_rows[4], ds.log_softmax_row(logits[2], 1.0), vocab_map)
    assert loss[0] == pytest.approx(l0) and loss[4] == pytest.approx(l4)
    # dynamic weight: the verified target probability of the n-gram
    loss2, _ = ds.distill_sequence(q_rows, d, [0, 1, 4], [1, 3, 1], 3, logits, 1.0, vocab_map, [d[0], 20, d[4]], 0.2,
                                   ds.LAMBDA_TARGET_PROB)
    w = np.exp(ds.log_softmax_row(logits[1], 1.0)[20])
    assert loss2[2] == pytest.approx(-w * np.log(q_rows[2, d[2]]))
