"""od_verify_noalloc, the step-2 entry point for callers that must not allocate
device memory (plug-ins living inside a process whose own allocator owns the
GPU's memory, loops that cannot take the synchronisation cudaMalloc implies).

It takes no context and keeps the kernels' scratch in a fixed array inside the
library. Checked here: called through the C ABI, it reproduces od_verify's outputs
on two calls in a row (different inputs: the array is reused with the previous
call's contents still in it); together with the translation and sampling steps of
a context it passes the full comparison with the CPU oracle; it works at the very
last row of its fixed array and with fp32 logits; and a call leaves the amount of
free device memory where it was.
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2507_02659_b200 import binding as od
from paper_2507_02659_b200 import synth

import parity

pytestmark = pytest.mark.gpu


def _workload(**kw):
    base = dict(B=8, steps=2, k_max=5, k_min=1, v_q=3000, v_p=20011,
                logit_dtype="bf16", map_kind="random", mapped_frac=0.7, cache_entries=500,
                hit_prob=0.6, logit_kind="corr", rho=0.95, temperatures=(1.0, 0.5, 0.7),
                per_seq_seed=True, gen_seed=0xBEEFA0, unmapped_shift=2.0, sigma=2.0)
    base.update(kw)
    return synth.Workload("noalloc", **base)


def _same_as_od_verify(got, ref, m):
    for b in range(len(m)):
        mb = int(m[b])
        # integer results and flags: identical
        assert int(got.n_accepted[b]) == int(ref.n_accepted[b])
        assert int(got.n_draft_accepted[b]) == int(ref.n_draft_accepted[b])
        assert int(got.flags[b]) == int(ref.flags[b])
        # floating point: the tolerances of the parity tests (rows 0..m_b, positions < m_b)
        assert torch.equal(got.row_max[b, :mb + 1], ref.row_max[b, :mb + 1])
        torch.testing.assert_close(got.row_sum[b, :mb + 1], ref.row_sum[b, :mb + 1], rtol=2e-5, atol=0)
        torch.testing.assert_close(got.p_sel[b, :mb], ref.p_sel[b, :mb], rtol=1e-5, atol=1e-30)
        torch.testing.assert_close(got.ratio[b, :mb], ref.ratio[b, :mb], rtol=0, atol=2e-5)


def test_noalloc_matches_od_verify_on_two_calls_in_a_row(cuda_device):
    torch.cuda.set_device(cuda_device)
    w = _workload()
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    B, K = w.B, w.k_max
    # everything the new entry point touches is allocated here, before it is called
    outs = [od.alloc_verify_out(ctx, B, K) for _ in range(2)]
    for step in range(2):
        s = synth.make_step(w, st, step, device=cuda_device)
        logits = parity.pad_rows(s.logits)          # 20011 ids: rows padded to 16-byte strides
        mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
        ref = od.od_verify(ctx, logits, mp, s.temperature, s.seed, step)
        got = od.od_verify_noalloc(w.v_p, logits, mp, s.temperature, s.seed, step, out=outs[step])
        torch.cuda.synchronize(cuda_device)
        m = mp.m.cpu().numpy()
        assert (m > 0).any()
        _same_as_od_verify(got, ref, m)
    ctx.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_step_matches_the_oracle_and_allocates_nothing(cuda_device, dtype):
    """Steps 1 and 3 from a context, step 2 from the allocation-free entry point: the whole step
    against the CPU oracle. Around the second call the free device memory must not move."""
    torch.cuda.set_device(cuda_device)
    w = _workload(B=12, logit_dtype=dtype, gen_seed=0xBEEFA1)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    vo = od.alloc_verify_out(ctx, w.B, w.k_max)
    for step in range(2):
        s = synth.make_step(w, st, step, device=cuda_device)
        logits = parity.pad_rows(s.logits)
        mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
        so = od.alloc_sample_out(ctx, w.B)
        torch.cuda.synchronize(cuda_device)
        free_before, _ = torch.cuda.mem_get_info(cuda_device)
        od.od_verify_noalloc(w.v_p, logits, mp, s.temperature, s.seed, step, out=vo)
        torch.cuda.synchronize(cuda_device)
        free_after, _ = torch.cuda.mem_get_info(cuda_device)
        if step == 1:                               # the first call may be where the driver loads the module
            assert free_after == free_before
        od.od_sample_residual(ctx, logits, vo, s.q_rows, s.draft_ids, mp, s.temperature, s.seed, step, out=so)
        torch.cuda.synchronize(cuda_device)
        ref = parity.oracle_step(cache, st, w, s.to("cpu"), probe=so.out_token.cpu().numpy())
        stats = parity.compare(mp, vo, so, ref, s.draft_len.cpu().numpy(), step,
                               s.seed.cpu().numpy().astype(np.uint64), bf16=(dtype == "bf16"))
        assert stats.sequences == w.B
    ctx.close()


def test_noalloc_at_the_last_row_of_its_array(cuda_device):
    """B * (K_max + 1) == OD_NOALLOC_MAX_ROWS: the call that fills the fixed array to its end."""
    torch.cuda.set_device(cuda_device)
    K = 7
    B = od.OD_NOALLOC_MAX_ROWS // (K + 1)
    assert B * (K + 1) == od.OD_NOALLOC_MAX_ROWS
    w = _workload(B=B, k_max=K, k_min=K, v_q=500, v_p=1203, cache_entries=0, hit_prob=0.0, mapped_frac=1.0,
                  unmapped_shift=0.0, gen_seed=0xBEEFA2)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 0, device=cuda_device)
    logits = parity.pad_rows(s.logits)
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    ref = od.od_verify(ctx, logits, mp, s.temperature, s.seed, 0)
    got = od.od_verify_noalloc(w.v_p, logits, mp, s.temperature, s.seed, 0, out=od.alloc_verify_out(ctx, B, K))
    torch.cuda.synchronize(cuda_device)
    m = mp.m.cpu().numpy()
    assert (m == K).any()                           # some sequence uses every row, the last of the array included
    _same_as_od_verify(got, ref, m)
    ctx.close()


def test_noalloc_refuses_what_its_scratch_cannot_hold(cuda_device):
    torch.cuda.set_device(cuda_device)
    dev = cuda_device
    K = 7
    B = od.OD_NOALLOC_MAX_ROWS // (K + 1) + 1        # one sequence too many
    z = lambda *s, dt=torch.int32: torch.zeros(*s, dtype=dt, device=dev)
    mp = od.MapOut(z(B, K), z(B, K, dt=torch.float32), z(B, K), z(B, K), z(B), z(B, dt=torch.uint8), z(4))
    out = od.VerifyOut(z(B, K + 1, dt=torch.float32), z(B, K + 1, dt=torch.float32), z(B, K, dt=torch.float32),
                       z(B, K, dt=torch.float32), z(B), z(B), z(B))
    logits = torch.zeros(B, K + 1, 64, dtype=torch.bfloat16, device=dev)
    T = torch.ones(B, device=dev)
    seed = torch.zeros(B, dtype=torch.int64, device=dev)
    with pytest.raises(od.OdError) as e:
        od.od_verify_noalloc(64, logits, mp, T, seed, 0, out=out)
    assert e.value.status == -9
    torch.cuda.synchronize(dev)
