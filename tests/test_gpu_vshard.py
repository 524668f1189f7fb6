"""Vocabulary-sharded verification: all shards of a step run one after the other on
one GPU through the C ABI (the calls a rank makes, in its order), and the combined
result is compared with the CPU oracle of the UNSHARDED step: splitting the columns
changes neither Algorithm 1 nor Eq. (2)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_02659_b200 import binding as od
from paper_2507_02659_b200 import synth, vshard

import parity

pytestmark = pytest.mark.gpu


def _workload(name, **kw):
    base = dict(B=24, steps=4, k_max=5, k_min=1, v_q=3000, v_p=5000, logit_dtype="bf16",
                map_kind="random", mapped_frac=0.7, cache_entries=600, hit_prob=0.6,
                logit_kind="corr", rho=0.95, temperatures=(1.0, 0.5, 0.7), per_seq_seed=True,
                gen_seed=0xBEEF90, unmapped_shift=2.0, sigma=2.0)
    base.update(kw)
    return synth.Workload(name, **base)


def _sharded_check(ctx, cache, st, w, s, n_shards, sel=None, copy_shards=False, logits=None):
    lg = s.logits if logits is None else logits
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    vo, so, picks = vshard.emulate_step(ctx, lg, n_shards, mp, s.q_rows, s.draft_ids, s.temperature,
                                        s.seed, s.step, copy_shards=copy_shards)
    torch.cuda.synchronize()
    # exactly one shard owns each token
    toks = torch.stack([p.out_token for p in picks])
    owners = (toks >= 0).sum(0)
    assert int(owners.max()) <= 1
    bounds = [vshard.split_vocab(w.v_p, r, n_shards) for r in range(n_shards)]
    for r, (lo, hi) in enumerate(bounds):
        t = toks[r][toks[r] >= 0]
        assert ((t >= lo) & (t < hi)).all()
    B = s.draft_ids.shape[0]
    idx = np.arange(B) if sel is None else np.asarray(sel)
    tix = torch.from_numpy(idx).to(s.draft_ids.device)
    pick = lambda t: t.index_select(0, tix).cpu()
    s_cpu = synth.StepInputs(pick(s.draft_ids), pick(s.draft_len), pick(s.q_sel), pick(s.q_rows),
                             pick(s.logits), pick(s.temperature), pick(s.seed), s.step)
    ref = parity.oracle_step(cache, st, w, s_cpu, probe=so.out_token.cpu().numpy()[idx])
    stats = parity.compare(mp, vo, so, ref, s_cpu.draft_len.numpy(), s.step,
                           s_cpu.seed.numpy().astype(np.uint64), bf16=(w.logit_dtype == "bf16"), sel=idx)
    return stats, (mp, vo, so)


@pytest.mark.parametrize("n_shards,dtype,copy", [(1, "bf16", False), (2, "bf16", False), (3, "f32", False),
                                                 (5, "bf16", True), (20, "f32", True)])
def test_sharded_step_matches_the_oracle(cuda_device, n_shards, dtype, copy):
    w = _workload(f"vs{n_shards}", logit_dtype=dtype, gen_seed=0xBEEF90 + n_shards)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    total = parity.Stats()
    for step in range(3):
        s = synth.make_step(w, st, step, device=cuda_device)
        stats, _ = _sharded_check(ctx, cache, st, w, s, n_shards, copy_shards=copy)
        total.merge(stats)
    assert total.sample_compared > 20 and total.cache_hits > 0 and total.unmapped_stops > 0
    ctx.close()


def test_sharded_step_with_colliding_cases_of_eq2(cuda_device):
    """Cached n-grams whose token has a direct pre-image, or is the image of the run's own first
    sub-token, rejected often enough that the sharded residual draw meets them."""
    w = _workload("vs_eq2", B=64, k_max=4, k_min=2, v_q=600, v_p=1000, cache_entries=400, hit_prob=0.95,
                  logit_kind="zipf", targets_in_image=0.4, targets_on_prefix=0.4, plant_boost=8.0,
                  gen_seed=0xBEEF9E)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    image = np.zeros(w.v_p, bool)
    image[st.vocab_map[st.vocab_map >= 0]] = True
    at_ngram_in_image = 0
    for step in range(4):
        s = synth.make_step(w, st, step, device=cuda_device)
        _, (mp, vo, so) = _sharded_check(ctx, cache, st, w, s, 3)
        m, n = mp.m.cpu().numpy(), vo.n_accepted.cpu().numpy()
        tgt, sl = mp.tgt_ids.cpu().numpy(), mp.span_len.cpu().numpy()
        for b in range(w.B):
            j = int(n[b])
            at_ngram_in_image += j < int(m[b]) and sl[b, j] >= 2 and bool(image[tgt[b, j]])
    assert at_ngram_in_image >= 20
    ctx.close()


def test_one_shard_is_bit_identical_to_the_unsharded_calls(cuda_device):
    w = _workload("vs1bits", B=40, v_p=9000)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 0, device=cuda_device)
    mp, vo, so = parity.gpu_step(ctx, s)
    vo2, so2 = vshard.step(ctx, 0, s.logits, mp, s.q_rows, s.draft_ids, s.temperature, s.seed, s.step)
    torch.cuda.synchronize()
    for a, b in ((vo.row_max, vo2.row_max), (vo.row_sum, vo2.row_sum), (vo.p_sel, vo2.p_sel),
                 (vo.ratio, vo2.ratio), (vo.n_accepted, vo2.n_accepted), (vo.flags, vo2.flags),
                 (so.out_token, so2.out_token), (so.resid_mass, so2.resid_mass), (so.flags, so2.flags)):
        m = mp.m.clamp(0, w.k_max)
        if a.dim() == 2:        # only rows / positions up to m_b are defined
            width = a.shape[1]
            keep = torch.arange(width, device=a.device)[None, :] < (m[:, None] + (1 if width == w.k_max + 1 else 0))
            assert torch.equal(a[keep], b[keep])
        else:
            assert torch.equal(a, b)
    ctx.close()


def test_shard_count_changes_decisions_only_at_flagged_boundaries(cuda_device):
    w = _workload("vsdet", B=64, v_p=20000, v_q=4000, gen_seed=0xBEEFA7)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 2, device=cuda_device)
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    ref_vo, ref_so, _ = vshard.emulate_step(ctx, s.logits, 1, mp, s.q_rows, s.draft_ids, s.temperature, s.seed, s.step)
    for n in (2, 7, 16):
        vo, so, _ = vshard.emulate_step(ctx, s.logits, n, mp, s.q_rows, s.draft_ids, s.temperature, s.seed, s.step)
        torch.cuda.synchronize()
        m = mp.m.clamp(0, w.k_max)
        keep = torch.arange(w.k_max + 1, device=m.device)[None, :] <= m[:, None]
        assert torch.equal(vo.row_max[keep], ref_vo.row_max[keep])            # maxima are exact
        assert torch.allclose(vo.row_sum[keep], ref_vo.row_sum[keep], rtol=2e-6)
        diff = vo.n_accepted != ref_vo.n_accepted
        assert ((vo.flags | ref_vo.flags)[diff] & od.OD_VF_BOUNDARY_MASK).ne(0).all()
        same = ~diff
        tdiff = same & (so.out_token != ref_so.out_token)
        assert ((so.flags | ref_so.flags)[tdiff] & od.OD_SF_BOUNDARY).ne(0).all()
    ctx.close()


def test_batched_128256_shape_eight_shards(cuda_device):
    """Config 4's launch (B = 64, 128256-id bf16 rows) split over 8 shards; the oracle
    recomputes a spread sample of the sequences."""
    w = synth.paper_config(4)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    s = synth.make_step(w, st, 0, device=cuda_device)
    sel = np.arange(0, 64, 3)
    stats, _ = _sharded_check(ctx, cache, st, w, s, 8, sel=sel)
    assert stats.sequences == len(sel) and stats.sample_compared > 0
    ctx.close()


def test_zero_residual_mass_on_every_shard_falls_back_to_p(cuda_device):
    """q' >= p on every id (uniform p, uniform q over the mapped ids): no shard has
    residual mass, so the token is drawn from p across the shards."""
    V = 1024
    ctx = od.Context(cuda_device, V + 1, V, 3, 1)
    vm = np.concatenate([np.arange(V, dtype=np.int32), np.array([-1], np.int32)])
    ctx.set_vocab_map(vm)
    empty = (np.zeros((0, 4), np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32))
    ctx.cache_build(*empty)
    dev = cuda_device
    logits = torch.zeros(3, 2, V, dtype=torch.float32, device=dev)
    q_rows = torch.zeros(3, 1, V + 1, dtype=torch.float32, device=dev)
    q_rows[:, 0, :V] = 1.0 / V
    d = torch.full((3, 1), V, dtype=torch.int32, device=dev)          # an unmapped id: forced rejection
    klen = torch.ones(3, dtype=torch.int32, device=dev)
    q_sel = torch.zeros(3, 1, dtype=torch.float32, device=dev)
    T = torch.ones(3, device=dev)
    seed = torch.arange(3, dtype=torch.int64, device=dev)
    mp = od.od_map_proposals(ctx, d, klen, q_sel)
    vo, so, picks = vshard.emulate_step(ctx, logits, 4, mp, q_rows, d, T, seed, 5)
    torch.cuda.synchronize()
    cache = oracle.Cache(*empty)
    ref = oracle.step_batch(cache, vm, V, d.cpu().numpy(), klen.cpu().numpy(), q_sel.cpu().numpy(),
                            q_rows.cpu().numpy(), np.zeros((3, 2, V), np.float32), oracle.DTYPE_F32,
                            np.ones(3, np.float32), np.arange(3, dtype=np.uint64), 5)
    for b in range(3):
        assert int(mp.tail_kind[b]) == od.OD_TAIL_UNMAPPED_STOP
        assert ref.flags[b] & oracle.FLAG_ZERO_MASS
        assert int(so.flags[b]) & od.OD_SF_ZERO_MASS
        assert int(so.out_token[b]) == int(ref.token[b])
        assert float(so.resid_mass[b]) == pytest.approx(1.0, abs=1e-6)
    ctx.close()


def test_bad_temperature_is_flagged_on_every_shard(cuda_device):
    w = _workload("vsbadT", B=4, temperatures=(1.0, 0.7, 0.9, 0.5))
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 0, device=cuda_device)
    s.temperature[1] = 0.0
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    vo, so, picks = vshard.emulate_step(ctx, s.logits, 3, mp, s.q_rows, s.draft_ids, s.temperature, s.seed, 0)
    torch.cuda.synchronize()
    assert int(vo.flags[1]) & od.OD_VF_BAD_TEMPERATURE and int(vo.n_accepted[1]) == 0
    assert int(so.flags[1]) & od.OD_SF_BAD_TEMPERATURE and int(so.out_token[1]) == -1
    assert int(so.out_token[0]) >= 0
    ctx.close()


def test_shard_arguments_are_validated(cuda_device):
    w = _workload("vsargs", B=2)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 0, device=cuda_device)
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    # a shard must start on a 256-id tile and end on one (or at the vocabulary's end)
    with pytest.raises(od.OdError) as e:
        od.od_verify_shard_stats(ctx, 128, s.logits[:, :, 128:1024].contiguous(), mp, s.temperature)
    assert e.value.status == od.OD_ERR_INVALID_ARG
    with pytest.raises(od.OdError) as e:
        od.od_verify_shard_stats(ctx, 256, s.logits[:, :, 256:1000].contiguous(), mp, s.temperature)
    assert e.value.status == od.OD_ERR_INVALID_ARG
    with pytest.raises(od.OdError) as e:
        od.od_verify_shard_stats(ctx, 4864, torch.zeros(2, w.k_max + 1, 512, dtype=torch.bfloat16, device=cuda_device),
                                 mp, s.temperature)                    # runs past the vocabulary
    assert e.value.status == od.OD_ERR_INVALID_ARG
    with pytest.raises(od.OdError):
        od.od_sample_shard_pick(ctx, 3, 0, torch.zeros(2, 2, 2, dtype=torch.float64, device=cuda_device),
                                s.logits[:, :, :256].contiguous(), od.alloc_verify_out(ctx, 2, w.k_max), s.q_rows,
                                s.draft_ids, mp, s.temperature, s.seed, 0)      # shard_index >= n_shards
    ctx.close()
