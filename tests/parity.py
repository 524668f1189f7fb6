"""Element-by-element comparison of the CUDA path with the CPU oracle.

Protocol (one verification step, B independent sequences):
  * mapping outputs (target ids, spans, m, tail kind, counters) are bit-exact;
    q' within 1e-6 relative (fp32 product against the fp64 product);
  * row maxima are exact, row sums within `sum_rtol`, p(t_i) and ratios within
    the absolute tolerance `p_atol` (1e-6 for fp32 logits, 2e-3 for bf16 logits
    are the bars; the achieved error is reported and asserted much tighter);
  * accept decisions: the GPU's decision at position i is u_i < ratio_i in fp32
    and can be replayed on the host from its own outputs; its prefix length
    must equal the leading accepts of that replay (exact), and every decision
    that differs from the oracle's fp64 decision must carry the GPU's boundary
    flag. A sequence is compared up to its first differing decision;
  * the extra token must equal the oracle's, or carry the boundary flag and be
    valid under the oracle's own fp64 CDF within the flag margin.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

import oracle
from paper_2507_02659_b200 import binding as od
from paper_2507_02659_b200 import synth


@dataclass
class Stats:
    sequences: int = 0
    decisions: int = 0
    accept_flagged: int = 0
    accept_mismatch_flagged: int = 0
    sample_compared: int = 0
    sample_flagged: int = 0
    sample_mismatch_flagged: int = 0
    degenerate: int = 0
    max_dp: float = 0.0
    max_dratio: float = 0.0
    max_dsum_rel: float = 0.0
    max_dmass: float = 0.0
    cache_hits: int = 0
    unmapped_stops: int = 0
    accepted: int = 0
    proposed: int = 0
    bonus: int = 0

    def merge(self, o: "Stats"):
        for k, v in o.__dict__.items():
            if k.startswith("max_"):
                setattr(self, k, max(getattr(self, k), v))
            else:
                setattr(self, k, getattr(self, k) + v)


def pad_rows(logits: torch.Tensor, multiple_bytes: int = 16) -> torch.Tensor:
    """A view [B, R, V] whose rows start on 16-byte boundaries (dense rows of an
    odd vocabulary do not)."""
    B, R, V = logits.shape
    per = multiple_bytes // logits.element_size()
    Vp = (V + per - 1) // per * per
    if Vp == V:
        return logits.contiguous()
    store = torch.full((B, R, Vp), float("nan"), dtype=logits.dtype, device=logits.device)
    store[:, :, :V] = logits
    return store[:, :, :V]


def make_context(w: synth.Workload, st: synth.Static, device, max_batch=None) -> od.Context:
    ctx = od.Context(device, w.v_q, w.v_p, max_batch or w.B, w.k_max)
    ctx.set_vocab_map(st.vocab_map)
    ctx.cache_build(st.runs, st.run_len, st.run_target)
    return ctx


def gpu_step(ctx: od.Context, s: synth.StepInputs, logits=None):
    """Runs the three C-ABI calls on device tensors; returns the output structs."""
    lg = s.logits if logits is None else logits
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    vo = od.od_verify(ctx, lg, mp, s.temperature, s.seed, s.step)
    so = od.od_sample_residual(ctx, lg, vo, s.q_rows, s.draft_ids, mp, s.temperature, s.seed, s.step)
    torch.cuda.synchronize(ctx.device)
    return mp, vo, so


def oracle_step(cache: oracle.Cache, st: synth.Static, w: synth.Workload, s_cpu: synth.StepInputs,
                probe=None, threads: int = 0) -> oracle.StepResult:
    lg, code = oracle.logits_to_numpy(s_cpu.logits)
    return oracle.step_batch(cache, st.vocab_map, w.v_p, s_cpu.draft_ids.numpy(),
                             s_cpu.draft_len.numpy(), s_cpu.q_sel.numpy(), s_cpu.q_rows.numpy(),
                             lg, code, s_cpu.temperature.numpy(),
                             s_cpu.seed.numpy().astype(np.uint64), s_cpu.step,
                             probe_token=probe, threads=threads)


def compare(mp, vo, so, ref: oracle.StepResult, draft_len, step: int, seeds, bf16: bool,
            sel=None, p_atol=None, sum_rtol=2e-5) -> Stats:
    """`sel`: indices of the GPU batch that `ref` covers (None = all)."""
    g = lambda t: t.detach().cpu().numpy()
    idx = np.arange(ref.m.shape[0]) if sel is None else np.asarray(sel)
    tgt, qp, ss, sl = g(mp.tgt_ids)[idx], g(mp.q_prime)[idx], g(mp.span_start)[idx], g(mp.span_len)[idx]
    m, tail = g(mp.m)[idx], g(mp.tail_kind)[idx]
    rmax, rsum = g(vo.row_max)[idx], g(vo.row_sum)[idx]
    psel, ratio = g(vo.p_sel)[idx], g(vo.ratio)[idx]
    nacc, ndr, vfl = g(vo.n_accepted)[idx], g(vo.n_draft_accepted)[idx], g(vo.flags)[idx].view(np.uint32)
    tok, mass, sfl = g(so.out_token)[idx], g(so.resid_mass)[idx], g(so.flags)[idx].view(np.uint32)
    if p_atol is None:
        p_atol = 2e-3 if bf16 else 1e-6
    st = Stats()
    B, K = tgt.shape
    st.sequences = B
    np.testing.assert_array_equal(m, ref.m)
    np.testing.assert_array_equal(tail.astype(np.int32), ref.tail_kind)
    for b in range(B):
        mb = int(m[b])
        np.testing.assert_array_equal(tgt[b, :mb], ref.tgt_ids[b, :mb])
        np.testing.assert_array_equal(sl[b, :mb], ref.span_len[b, :mb])
        ns = mb + (1 if tail[b] == od.OD_TAIL_UNMAPPED_STOP else 0)
        np.testing.assert_array_equal(ss[b, :ns], ref.span_start[b, :ns])
        np.testing.assert_allclose(qp[b, :mb], ref.q_prime[b, :mb], rtol=1e-6, atol=1e-37)
        st.cache_hits += int(ref.hits[b])
        st.unmapped_stops += int(tail[b] == od.OD_TAIL_UNMAPPED_STOP)
        st.proposed += int(draft_len[b])
        if ref.flags[b] & oracle.FLAG_BAD_TEMPERATURE:
            assert vfl[b] & od.OD_VF_BAD_TEMPERATURE and sfl[b] & od.OD_SF_BAD_TEMPERATURE
            assert nacc[b] == 0 and tok[b] == -1
            continue
        assert not (vfl[b] & (od.OD_VF_BAD_TEMPERATURE | od.OD_VF_NONFINITE)), hex(vfl[b])
        # row statistics, rows 0..m
        assert (rmax[b, :mb + 1].astype(np.float64) == ref.row_max[b, :mb + 1]).all(), (b, rmax[b], ref.row_max[b])
        rel = np.abs(rsum[b, :mb + 1] / ref.row_sum[b, :mb + 1] - 1.0).max()
        st.max_dsum_rel = max(st.max_dsum_rel, float(rel))
        assert rel <= sum_rtol, (b, rel)
        if mb:
            dp = np.abs(psel[b, :mb] - ref.p_sel[b, :mb]).max()
            dr = np.abs(ratio[b, :mb] - ref.ratio[b, :mb]).max()
            st.max_dp = max(st.max_dp, float(dp)); st.max_dratio = max(st.max_dratio, float(dr))
            assert dp <= p_atol, (b, dp)
            # relative check as well: fp32 arithmetic on identical inputs
            relp = np.abs(psel[b, :mb] - ref.p_sel[b, :mb]) / np.maximum(ref.p_sel[b, :mb], 1e-30)
            assert (relp[ref.p_sel[b, :mb] > 1e-12] <= 1e-5).all(), (b, relp)
            assert dr <= max(p_atol, 2e-5), (b, dr)
        # replay the GPU's decisions from its own ratios
        u = np.array([np.float32(oracle.uniform(int(seeds[b]), step, i, 0)) for i in range(mb)], np.float32)
        np.testing.assert_array_equal(u.astype(np.float64), ref.u_acc[b, :mb])
        acc_gpu = u < ratio[b, :mb]
        lead = 0
        while lead < mb and acc_gpu[lead]:
            lead += 1
        assert nacc[b] == lead, (b, nacc[b], lead)
        assert ndr[b] == int(sl[b, :lead].sum())
        bflags = np.array([(vfl[b] >> i) & 1 for i in range(mb)], bool)
        near = np.abs(u.astype(np.float64) - ratio[b, :mb].astype(np.float64)) <= od.OD_TAU_ACCEPT * (1 - 1e-3)
        assert (bflags[near]).all(), (b, "a decision inside the margin is not flagged")
        cut = False
        for i in range(mb):
            st.decisions += 1
            st.accept_flagged += int(bflags[i])
            if bool(acc_gpu[i]) != bool(ref.accept[b, i]):
                assert bflags[i], (b, i, u[i], ratio[b, i], ref.ratio[b, i], "unflagged accept mismatch")
                st.accept_mismatch_flagged += 1
                cut = True
                break
            if not acc_gpu[i]:
                break
        if cut:
            continue
        assert nacc[b] == ref.n_accepted[b]
        assert ndr[b] == ref.n_draft_accepted[b]
        st.accepted += int(nacc[b])
        # extra token
        gpu_bonus = bool(sfl[b] & od.OD_SF_BONUS)
        assert gpu_bonus == (ref.kind[b] == oracle.KIND_BONUS), (b, sfl[b], ref.kind[b])
        st.bonus += int(gpu_bonus)
        zero_g = bool(sfl[b] & od.OD_SF_ZERO_MASS)
        zero_o = bool(ref.flags[b] & oracle.FLAG_ZERO_MASS)
        if zero_g != zero_o:
            # a residual mass that is zero on one side must be negligible on the other
            assert min(float(mass[b]), float(ref.mass[b])) <= 1e-5 or zero_g and float(ref.mass[b]) <= 1e-5 \
                or zero_o and float(mass[b]) <= 1e-5, (b, mass[b], ref.mass[b])
            st.degenerate += 1
            continue
        dm = abs(float(mass[b]) - float(ref.mass[b]))
        st.max_dmass = max(st.max_dmass, dm)
        assert dm <= max(p_atol, 1e-5) , (b, mass[b], ref.mass[b])
        st.sample_compared += 1
        flagged = bool(sfl[b] & od.OD_SF_BOUNDARY)
        st.sample_flagged += int(flagged)
        assert 0 <= tok[b] < 2**31
        R = float(ref.mass[b])
        target = float(ref.u_samp[b]) * R
        if tok[b] != ref.token[b]:
            assert flagged, (b, tok[b], ref.token[b], "unflagged token mismatch")
            st.sample_mismatch_flagged += 1
        # valid under the oracle's CDF within the margin, equal or not
        tau = 2.0 * od.OD_TAU_SAMPLE * R
        assert ref.probe_lo[b] - tau <= target <= ref.probe_hi[b] + tau, \
            (b, tok[b], ref.token[b], ref.probe_lo[b], target, ref.probe_hi[b])
        assert ref.probe_hi[b] > ref.probe_lo[b], (b, "token without residual mass")
    return st


def check_step(ctx, cache, st, w, s_dev: synth.StepInputs, sel=None, threads=0, logits=None, **kw) -> Stats:
    """GPU step on `s_dev`, oracle on the same bytes (optionally only on the
    sequences `sel`), full comparison."""
    mp, vo, so = gpu_step(ctx, s_dev, logits=logits)
    B = s_dev.draft_ids.shape[0]
    idx = np.arange(B) if sel is None else np.asarray(sel)
    tix = torch.from_numpy(idx).to(s_dev.draft_ids.device)
    pick = lambda t: t.index_select(0, tix).cpu()
    s_cpu = synth.StepInputs(pick(s_dev.draft_ids), pick(s_dev.draft_len), pick(s_dev.q_sel),
                             pick(s_dev.q_rows), pick(s_dev.logits), pick(s_dev.temperature),
                             pick(s_dev.seed), s_dev.step)
    probe = so.out_token.detach().cpu().numpy()[idx]
    ref = oracle_step(cache, st, w, s_cpu, probe=probe, threads=threads)
    return compare(mp, vo, so, ref, s_cpu.draft_len.numpy(), s_dev.step,
                   s_cpu.seed.numpy().astype(np.uint64), bf16=(w.logit_dtype == "bf16"), sel=idx, **kw)
