"""GPU parity of the hybrid distillation loss (Eq. (3)) and its gradient with the fp64
oracle, on the translated proposals of real verification steps."""
import numpy as np
import pytest
import torch

import oracle
from oracle import distill as ds
from paper_2507_02659_b200 import binding as od
from paper_2507_02659_b200 import synth

import parity

pytestmark = pytest.mark.gpu


def _logits64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _check(w, device, steps, lam, mode, positions=None):
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, device)
    seen = {"kl": 0, "nll": 0, "none": 0}
    for step in steps:
        s = synth.make_step(w, st, step, device=device)
        logits = parity.pad_rows(s.logits)
        mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
        vo = od.od_verify(ctx, logits, mp, s.temperature, s.seed, step)
        loss, grad = od.od_distill_loss(ctx, s.q_rows, s.draft_ids, mp, logits, vo, s.temperature, lam, mode)
        torch.cuda.synchronize()
        m = mp.m.cpu().numpy(); ss = mp.span_start.cpu().numpy(); sl = mp.span_len.cpu().numpy()
        tg = mp.tgt_ids.cpu().numpy(); d = s.draft_ids.cpu().numpy(); T = s.temperature.cpu().numpy()
        loss, grad = loss.cpu().numpy(), grad.cpu().numpy()
        seqs = range(w.B) if positions is None else positions
        for b in seqs:
            q_rows = s.q_rows[b].cpu().numpy().astype(np.float64)
            want_l, want_g = ds.distill_sequence(q_rows, d[b], ss[b], sl[b], m[b], _logits64(s.logits[b]),
                                                 float(T[b]), st.vocab_map, tg[b], lam, mode)
            np.testing.assert_allclose(loss[b], want_l, rtol=2e-5, atol=2e-6)
            np.testing.assert_allclose(grad[b], want_g, rtol=1e-4, atol=2e-6)
            for i in range(int(m[b])):
                seen["kl" if sl[b, i] == 1 else "nll"] += int(sl[b, i])
            covered = int(sl[b, :m[b]].sum())
            seen["none"] += w.k_max - covered
            assert not grad[b, covered:].any() and not loss[b, covered:].any()
    ctx.close()
    return seen


def _small(**kw):
    base = dict(B=6, steps=4, k_max=5, k_min=1, v_q=600, v_p=1000, logit_dtype="bf16", map_kind="random",
                mapped_frac=0.7, cache_entries=300, hit_prob=0.7, logit_kind="corr", rho=0.95,
                temperatures=(1.0, 0.5, 0.7), per_seq_seed=True, gen_seed=0xBEEFD0, unmapped_shift=2.0, sigma=2.0)
    base.update(kw)
    return synth.Workload("distill", **base)


@pytest.mark.parametrize("mode", [ds.LAMBDA_CONSTANT, ds.LAMBDA_TARGET_PROB])
def test_loss_and_gradient_match_the_oracle(cuda_device, mode):
    seen = _check(_small(B=12), cuda_device, range(4), 0.2, mode)
    assert seen["kl"] > 20 and seen["nll"] > 10 and seen["none"] > 10


def test_fp32_logits_and_odd_vocabularies(cuda_device):
    _check(_small(v_q=333, v_p=1003, logit_dtype="f32", cache_entries=100, gen_seed=0xBEEFD1), cuda_device,
           range(3), 0.2, ds.LAMBDA_CONSTANT)


def test_full_vocabulary_sampled_sequences(cuda_device):
    """The batched 128256-id shape; the oracle recomputes a few sequences."""
    w = synth.scaled(synth.paper_config(4), B=16, name="cfg4-distill")
    _check(w, cuda_device, [0], 0.2, ds.LAMBDA_CONSTANT, positions=[0, 5, 11])


@pytest.mark.parametrize("i", range(8))
def test_random_shapes(cuda_device, i):
    """Seeded random vocabulary sizes (both the 128-bit path, V_q a multiple of 4, and the scalar one),
    proposal lengths, maps and temperatures."""
    rng = np.random.default_rng(7000 + i)
    v_q = int(rng.integers(50, 2500))
    if i % 2 == 0:
        v_q = v_q // 4 * 4
    v_p = int(rng.integers(v_q, 5000))
    k_max = int(rng.integers(1, 9))
    w = _small(B=int(rng.integers(1, 12)), k_max=k_max, k_min=int(rng.integers(1, k_max + 1)), v_q=v_q, v_p=v_p,
               logit_dtype=["bf16", "f32"][int(rng.integers(0, 2))], mapped_frac=float(rng.uniform(0.3, 0.9)),
               cache_entries=int(rng.integers(0, 200)), gen_seed=0xBEEFE0 + i)
    _check(w, cuda_device, range(2), lam=float(rng.uniform(0.05, 1.0)), mode=int(rng.integers(0, 2)))


@pytest.mark.parametrize("v_q", [600, 333])
def test_loss_without_a_gradient_buffer(cuda_device, v_q):
    """grad = NULL: the kernel has nowhere to park q*g between its sweeps and recomputes it; the
    loss must be the oracle's all the same (vector path for V_q = 600, scalar path for 333)."""
    w = _small(B=10, v_q=v_q, v_p=1003, cache_entries=150, gen_seed=0xBEEFD7)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    for step in range(3):
        s = synth.make_step(w, st, step, device=cuda_device)
        logits = parity.pad_rows(s.logits)
        mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
        vo = od.od_verify(ctx, logits, mp, s.temperature, s.seed, step)
        loss, grad = od.od_distill_loss(ctx, s.q_rows, s.draft_ids, mp, logits, vo, s.temperature, 0.2,
                                        ds.LAMBDA_CONSTANT, want_grad=False)
        with_grad, _ = od.od_distill_loss(ctx, s.q_rows, s.draft_ids, mp, logits, vo, s.temperature, 0.2,
                                          ds.LAMBDA_CONSTANT)
        torch.cuda.synchronize()
        assert grad is None
        m = mp.m.cpu().numpy(); ss = mp.span_start.cpu().numpy(); sl = mp.span_len.cpu().numpy()
        tg = mp.tgt_ids.cpu().numpy(); d = s.draft_ids.cpu().numpy(); T = s.temperature.cpu().numpy()
        loss = loss.cpu().numpy()
        for b in range(w.B):
            want_l, _ = ds.distill_sequence(s.q_rows[b].cpu().numpy().astype(np.float64), d[b], ss[b], sl[b], m[b],
                                            _logits64(s.logits[b]), float(T[b]), st.vocab_map, tg[b], 0.2,
                                            ds.LAMBDA_CONSTANT)
            np.testing.assert_allclose(loss[b], want_l, rtol=2e-5, atol=2e-6)
        np.testing.assert_allclose(loss, with_grad.cpu().numpy(), rtol=1e-6, atol=1e-7)
    ctx.close()
