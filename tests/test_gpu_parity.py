"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_02659_b200 import binding as od
from paper_2507_02659_b200 import synth

import parity

pytestmark = pytest.mark.gpu


def _small(name, **kw):
    base = dict(B=6, steps=4, k_max=5, k_min=1, v_q=600, v_p=1000, logit_dtype="bf16",
                map_kind="random", mapped_frac=0.7, cache_entries=300, hit_prob=0.6,
                logit_kind="corr", rho=0.95, temperatures=(1.0, 0.5, 0.7), per_seq_seed=True,
                gen_seed=0xBEEF00, unmapped_shift=2.0, sigma=2.0)
    base.update(kw)
    return synth.Workload(name, **base)


def _run_workload(w, device, steps, pad=False, opts=None, sel=None, **kw):
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, device)
    for k, v in (opts or {}).items():
        ctx.set_option(k, v)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    total = parity.Stats()
    for step in steps:
        s = synth.make_step(w, st, step, device=device)
        lg = parity.pad_rows(s.logits) if pad else None
        total.merge(parity.check_step(ctx, cache, st, w, s, logits=lg, sel=sel, **kw))
    ctx.close()
    return total


def _assert_rates(s: parity.Stats, max_accept_flag_rate=2e-3):
    if s.decisions >= 1000:
        assert s.accept_flagged <= max(3, max_accept_flag_rate * s.decisions), s
    assert s.sample_compared > 0


# ------------------------------------------------------------ tiny shapes
@pytest.mark.parametrize("v_p,dtype", [(8, "f32"), (8, "bf16"), (33, "bf16"), (33, "f32"),
                                        (1000, "bf16"), (1003, "f32"), (4099, "bf16")])
def test_tiny_vocabularies_and_ragged_tails(cuda_device, v_p, dtype):
    v_q = min(v_p, 600)
    w = _small(f"tiny{v_p}{dtype}", v_q=v_q, v_p=v_p, logit_dtype=dtype,
               mapped_frac=0.6 if v_p > 8 else 0.75,
               cache_entries=0 if v_p <= 8 else 100, gen_seed=0xBEEF00 + v_p)
    s = _run_workload(w, cuda_device, range(6), pad=True)
    assert s.sequences == 36


@pytest.mark.parametrize("T", [0.01, 0.5, 1.0])
def test_temperatures(cuda_device, T):
    w = _small(f"T{T}", temperatures=(T,), B=16, gen_seed=0xBEEF10)
    s = _run_workload(w, cuda_device, range(4))
    assert s.decisions > 0


def test_identity_map_fp32_high_acceptance(cuda_device):
    w = _small("ident", map_kind="identity", v_q=2000, v_p=2000, logit_dtype="f32", cache_entries=0,
               hit_prob=0.0, logit_kind="noise", B=32, k_max=6, k_min=6, temperatures=(1.0,),
               gen_seed=0xBEEF20)
    s = _run_workload(w, cuda_device, range(8))
    assert s.accepted > 0.3 * s.proposed          # exercises long prefixes and the bonus branch
    assert s.bonus > 0
    assert s.max_dp <= 1e-6


def test_cache_hits_and_unmapped_stops_are_exercised(cuda_device):
    w = _small("hits", B=64, hit_prob=0.9, gen_seed=0xBEEF30)
    s = _run_workload(w, cuda_device, range(4))
    assert s.cache_hits > 50 and s.unmapped_stops > 5


def _eq2_collision_counts(w, st, s, mp, vo):
    """How many sequences of the step draw their extra token at a cached n-gram whose target
    (a) has a direct pre-image of its own, (b) is the image of the run's first sub-token."""
    image = np.zeros(w.v_p, bool)
    image[st.vocab_map[st.vocab_map >= 0]] = True
    m, n = mp.m.cpu().numpy(), vo.n_accepted.cpu().numpy()
    tgt, sl, ss = mp.tgt_ids.cpu().numpy(), mp.span_len.cpu().numpy(), mp.span_start.cpu().numpy()
    d = s.draft_ids.cpu().numpy()
    inside = prefix = 0
    for b in range(w.B):
        j = int(n[b])
        if j < int(m[b]) and sl[b, j] >= 2:
            T = int(tgt[b, j])
            on_prefix = int(st.vocab_map[d[b, ss[b, j]]]) == T
            prefix += on_prefix
            inside += bool(image[T]) and not on_prefix
    return inside, prefix


def test_eq2_collisions_cache_targets_inside_the_image(cuda_device):
    """Eq. (2) when its cases collide: cached n-grams whose token has a direct pre-image, or is the
    image of the run's own first sub-token. The residual of such a position must use the n-gram's
    probability at that token (the oracle's reading, pinned by hand-worked vectors)."""
    w = _small("eq2col", B=96, k_max=4, k_min=2, hit_prob=0.95, cache_entries=400, targets_in_image=0.4,
               targets_on_prefix=0.4, plant_boost=8.0, logit_kind="zipf", gen_seed=0xBEEF35)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    inside = prefix = 0
    total = parity.Stats()
    for step in range(6):
        s = synth.make_step(w, st, step, device=cuda_device)
        mp, vo, so = parity.gpu_step(ctx, s)
        ref = parity.oracle_step(cache, st, w, s.to("cpu"), probe=so.out_token.cpu().numpy())
        total.merge(parity.compare(mp, vo, so, ref, s.draft_len.cpu().numpy(), s.step,
                                   s.seed.cpu().numpy().astype(np.uint64), bf16=True))
        a, b = _eq2_collision_counts(w, st, s, mp, vo)
        inside += a; prefix += b
    ctx.close()
    assert total.cache_hits > 100
    assert inside >= 30 and prefix >= 30, (inside, prefix)


@pytest.mark.parametrize("grid,tiles,pdl,early", [(1, 1, 1, 0), (2, 2, 0, 0), (7, 7, 1, 1), (37, 1000, 0, 1),
                                                  (0, 5, 1, 1), (400, 3, 1, 0)])
def test_every_split_of_a_row_gives_the_same_answer(cuda_device, grid, tiles, pdl, early):
    w = _small("split", v_q=3000, v_p=20011, B=5, cache_entries=500, gen_seed=0xBEEF40)
    _run_workload(w, cuda_device, range(3), pad=True,
                  opts={"verify_grid": grid, "sample_tiles_per_warp": tiles, "pdl": pdl, "early_inputs": early})


@pytest.mark.parametrize("grid,pdl,early", [(1, 1, 1), (3, 0, 0), (0, 1, 1), (101, 1, 0)])
def test_every_split_of_a_long_row_gives_the_same_answer(cuda_device, grid, pdl, early):
    """Rows of 128 KB and more are streamed by blocks of 16 warps (16 partials per block segment):
    70001 bf16 ids are 274 units of 512 bytes, the last one ragged."""
    w = _small("splitwide", v_q=3000, v_p=70001, B=4, cache_entries=500, gen_seed=0xBEEF41)
    _run_workload(w, cuda_device, range(2), pad=True, opts={"verify_grid": grid, "pdl": pdl, "early_inputs": early})


def test_sampler_tile_sums_on_the_batched_shape(cuda_device):
    """Pass 1 of the sampler (sums of e minus the list corrections) on 128256-id rows."""
    w = synth.scaled(synth.paper_config(4), B=48, gen_seed=0xBEEF49)
    _run_workload(w, cuda_device, [0], sel=np.arange(0, 48, 4))


def test_max_k_and_zero_length_proposals(cuda_device):
    w = _small("k16", k_max=16, k_min=0, B=40, v_q=500, v_p=700, cache_entries=200, hit_prob=0.8,
               unmapped_shift=6.0, gen_seed=0xBEEF50)
    s = _run_workload(w, cuda_device, range(4), pad=True)
    assert s.sequences == 160


def test_batches_beyond_one_verify_launch(cuda_device):
    """od_verify handles at most 2048 sequences per launch and goes through longer batches in
    slices: sequences on both sides of the cut are compared with the oracle."""
    w = _small("slices", B=2500, v_q=300, v_p=777, cache_entries=100, gen_seed=0xBEEF55)
    sel = np.concatenate([np.arange(0, 2500, 97), np.arange(2040, 2056), np.array([2499])])
    s = _run_workload(w, cuda_device, [0], pad=True, sel=np.unique(sel))
    assert s.sequences == len(np.unique(sel))


# ------------------------------------------------------------ the five configs
def test_config1_full_shape(cuda_device):
    w = synth.paper_config(1)
    s = _run_workload(w, cuda_device, range(40))
    assert s.max_dp <= 1e-6
    _assert_rates(s)


def test_config2_full_shape(cuda_device):
    s = _run_workload(synth.paper_config(2), cuda_device, range(12))
    assert s.max_dp <= 2e-3
    _assert_rates(s)


def test_config3_full_shape(cuda_device):
    s = _run_workload(synth.paper_config(3), cuda_device, range(12))
    _assert_rates(s)


def test_config4_full_batch(cuda_device):
    s = _run_workload(synth.paper_config(4), cuda_device, range(3))
    assert s.sequences == 192
    _assert_rates(s)


def test_config5_full_batch_sampled_sequences(cuda_device):
    """The launch the benchmark sweep uses (B = 512, 152064-id rows); the oracle
    recomputes a spread sample of the sequences one by one."""
    w = synth.paper_config(5)
    sel = np.arange(0, 512, 11)
    s = _run_workload(w, cuda_device, [0], sel=sel)
    assert s.sequences == len(sel)
    _assert_rates(s)


def test_same_vocabulary_ragged_batch_sampled_sequences(cuda_device):
    """Workload 6: 256 sequences, identity map over 32000 ids, no cache, ragged K."""
    w = synth.paper_config(6)
    sel = np.arange(0, 256, 3)
    s = _run_workload(w, cuda_device, [0, 1], sel=sel)
    assert s.sequences == 2 * len(sel)
    assert s.cache_hits == 0 and s.unmapped_stops == 0
    _assert_rates(s)


# ------------------------------------------------------------ properties
def test_results_are_bit_identical_run_to_run(cuda_device):
    w = _small("det", B=48, v_q=3000, v_p=50000, cache_entries=1000, gen_seed=0xBEEF60)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 0, device=cuda_device)
    outs = []
    for _ in range(3):
        mp, vo, so = parity.gpu_step(ctx, s)
        outs.append([t.clone() for t in (mp.tgt_ids, mp.q_prime, vo.row_max, vo.row_sum, vo.p_sel,
                                         vo.ratio, vo.n_accepted, vo.flags, so.out_token,
                                         so.resid_mass, so.flags)])
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a, b)
    ctx.close()


def test_sampling_directly_after_the_translation_gives_the_same_token(cuda_device):
    """od_sample_residual prepares its positions before it waits for the kernel in front of it;
    directly behind od_map_proposals (whose outputs it reads) it must not."""
    w = _small("mapsample", B=64, v_q=3000, v_p=40000, cache_entries=1000, gen_seed=0xBEEF65)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 0, device=cuda_device)
    mp, vo, so = parity.gpu_step(ctx, s)
    for _ in range(5):
        mp2 = od.alloc_map_out(ctx, w.B, w.k_max)
        for t in (mp2.tgt_ids, mp2.span_start, mp2.span_len, mp2.m):
            t.fill_(-1)                                  # whatever is read too early is wrong
        torch.cuda.synchronize()
        od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel, out=mp2)
        so2 = od.od_sample_residual(ctx, s.logits, vo, s.q_rows, s.draft_ids, mp2, s.temperature, s.seed, s.step)
        torch.cuda.synchronize()
        assert torch.equal(so2.out_token, so.out_token) and torch.equal(so2.flags, so.flags)
        assert torch.equal(so2.resid_mass, so.resid_mass)
    ctx.close()


def test_a_producer_directly_in_front_of_the_step_is_safe(cuda_device):
    """The logits are written by the launch directly in front of the library's first kernel (as a
    target model's output layer would), over rows that held NaN until then. With the default
    options nothing may be read before that launch has finished: od_step (whose streaming kernel
    starts on rows 0 early, behind its own translation kernel), od_verify on its own, and
    od_verify_noalloc must all match the oracle, every time."""
    w = _small("producer", B=48, v_q=3000, v_p=40000, cache_entries=1000, gen_seed=0xBEEF66)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    s = synth.make_step(w, st, 0, device=cuda_device)
    clean = s.logits.clone()
    temps = s.temperature.clone()
    ref = None
    for rep in range(20):
        which = rep % 3
        mp = od.alloc_map_out(ctx, w.B, w.k_max)
        if which != 0:
            od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel, out=mp)
        vo = od.alloc_verify_out(ctx, w.B, w.k_max)
        so = od.alloc_sample_out(ctx, w.B)
        s.logits.fill_(float("nan"))
        s.temperature.fill_(float("nan"))
        torch.cuda.synchronize()
        s.temperature.copy_(temps)
        s.logits.copy_(clean)                       # the producer: the launch directly in front
        if which == 0:
            od.od_step(ctx, s.draft_ids, s.draft_len, s.q_sel, s.q_rows, s.logits, s.temperature, s.seed, s.step,
                       mp=mp, vo=vo, so=so)
        else:
            if which == 1:
                od.od_verify(ctx, s.logits, mp, s.temperature, s.seed, s.step, out=vo)
            else:
                od.od_verify_noalloc(w.v_p, s.logits, mp, s.temperature, s.seed, s.step, out=vo)
            od.od_sample_residual(ctx, s.logits, vo, s.q_rows, s.draft_ids, mp, s.temperature, s.seed, s.step, out=so)
        torch.cuda.synchronize()
        if ref is None:
            ref = parity.oracle_step(cache, st, w, s.to("cpu"), probe=so.out_token.cpu().numpy())
            first = [t.clone() for t in (vo.row_sum, vo.n_accepted, so.out_token)]
        parity.compare(mp, vo, so, ref, s.draft_len.cpu().numpy(), s.step,
                       s.seed.cpu().numpy().astype(np.uint64), bf16=True)
        assert torch.equal(vo.n_accepted, first[1]) and torch.equal(so.out_token, first[2])
    ctx.close()


def test_a_producer_that_releases_its_dependents_before_it_writes(cuda_device):
    """The launch directly in front of the library's first kernel is a kernel that executes
    griddepcontrol.launch_dependents first and writes the logits (over NaN) half a millisecond
    later, as an output-layer GEMM built for programmatic dependent launch does, only slower: the
    library's kernels are resident and past their prologues long before the logits exist.
    With the default options every library kernel that reads the logits must still see them:
    od_step, od_verify on its own and od_verify_noalloc against the oracle, every time."""
    import helpers
    prod = helpers.early_producer_lib()
    w = _small("earlyproducer", B=48, v_q=3000, v_p=40000, cache_entries=1000, gen_seed=0xBEEF68)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    s = synth.make_step(w, st, 0, device=cuda_device)
    clean = s.logits.clone()
    nbytes = clean.numel() * clean.element_size()
    assert nbytes % 16 == 0
    stream = torch.cuda.current_stream(cuda_device).cuda_stream
    ref = None
    for rep in range(18):
        which = rep % 3
        mp = od.alloc_map_out(ctx, w.B, w.k_max)
        if which != 0:
            od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel, out=mp)
        vo = od.alloc_verify_out(ctx, w.B, w.k_max)
        so = od.alloc_sample_out(ctx, w.B)
        s.logits.fill_(float("nan"))
        torch.cuda.synchronize()
        assert prod.early_producer(s.logits.data_ptr(), clean.data_ptr(), nbytes, 1000000, stream) == 0
        if which == 0:
            od.od_step(ctx, s.draft_ids, s.draft_len, s.q_sel, s.q_rows, s.logits, s.temperature, s.seed, s.step,
                       mp=mp, vo=vo, so=so)
        else:
            if which == 1:
                od.od_verify(ctx, s.logits, mp, s.temperature, s.seed, s.step, out=vo)
            else:
                od.od_verify_noalloc(w.v_p, s.logits, mp, s.temperature, s.seed, s.step, out=vo)
            od.od_sample_residual(ctx, s.logits, vo, s.q_rows, s.draft_ids, mp, s.temperature, s.seed, s.step, out=so)
        torch.cuda.synchronize()
        if ref is None:
            ref = parity.oracle_step(cache, st, w, s.to("cpu"), probe=so.out_token.cpu().numpy())
        parity.compare(mp, vo, so, ref, s.draft_len.cpu().numpy(), s.step,
                       s.seed.cpu().numpy().astype(np.uint64), bf16=True)
    ctx.close()


def test_od_step_equals_the_three_calls(cuda_device):
    w = _small("onecall", B=40, v_q=3000, v_p=30011, cache_entries=800, gen_seed=0xBEEF67)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    s = synth.make_step(w, st, 3, device=cuda_device)
    lg = parity.pad_rows(s.logits)
    mp, vo, so = parity.gpu_step(ctx, s, logits=lg)
    mp2, vo2, so2 = od.od_step(ctx, s.draft_ids, s.draft_len, s.q_sel, s.q_rows, lg, s.temperature, s.seed, s.step)
    torch.cuda.synchronize()
    m = mp.m.clamp(0, w.k_max)
    rows = torch.arange(w.k_max + 1, device=cuda_device)[None, :] <= m[:, None]
    pos = torch.arange(w.k_max, device=cuda_device)[None, :] < m[:, None]
    assert torch.equal(mp.m, mp2.m) and torch.equal(mp.tgt_ids[pos], mp2.tgt_ids[pos])
    assert torch.equal(mp.tail_kind, mp2.tail_kind) and torch.equal(mp.counters, mp2.counters)
    assert torch.equal(vo.row_sum[rows], vo2.row_sum[rows]) and torch.equal(vo.row_max[rows], vo2.row_max[rows])
    assert torch.equal(vo.p_sel[pos], vo2.p_sel[pos]) and torch.equal(vo.ratio[pos], vo2.ratio[pos])
    assert torch.equal(vo.n_accepted, vo2.n_accepted) and torch.equal(vo.n_draft_accepted, vo2.n_draft_accepted)
    assert torch.equal(vo.flags, vo2.flags)
    assert torch.equal(so.out_token, so2.out_token) and torch.equal(so.flags, so2.flags)
    assert torch.equal(so.resid_mass, so2.resid_mass)
    # inputs that have been resident since a synchronisation: the caller may promise so
    # ("early_inputs"), and then the translation kernel reads the proposal before it waits
    # for the sampler of the step in front. Steps back to back, same bits.
    ctx.set_option("early_inputs", 1)
    torch.cuda.synchronize()
    runs = [od.od_step(ctx, s.draft_ids, s.draft_len, s.q_sel, s.q_rows, lg, s.temperature, s.seed, s.step)
            for _ in range(6)]
    torch.cuda.synchronize()
    for mp3, vo3, so3 in runs:
        assert torch.equal(mp.m, mp3.m) and torch.equal(mp.tgt_ids[pos], mp3.tgt_ids[pos])
        assert torch.equal(mp.q_prime[pos], mp3.q_prime[pos]) and torch.equal(mp.tail_kind, mp3.tail_kind)
        assert torch.equal(vo.row_sum[rows], vo3.row_sum[rows]) and torch.equal(vo.n_accepted, vo3.n_accepted)
        assert torch.equal(so.out_token, so3.out_token) and torch.equal(so.resid_mass, so3.resid_mass)
    ctx.close()


def test_rows_above_m_are_never_read(cuda_device):
    """Rows m_b+1.. hold NaN: any touch would poison the sums."""
    w = _small("nan", B=32, gen_seed=0xBEEF70)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    s = synth.make_step(w, st, 1, device=cuda_device)
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    m = mp.m.cpu().numpy()
    assert (m < w.k_max).any()
    for b in range(w.B):
        s.logits[b, m[b] + 1:] = float("nan")
    # positions >= K_b of the proposal are padding as well
    for b in range(w.B):
        kb = int(s.draft_len[b])
        s.draft_ids[b, kb:] = -7
        s.q_sel[b, kb:] = float("nan")
    ref_inputs = synth.StepInputs(s.draft_ids, s.draft_len, s.q_sel, s.q_rows,
                                  torch.nan_to_num(s.logits.float(), nan=0.0).to(s.logits.dtype),
                                  s.temperature, s.seed, s.step)
    mp, vo, so = parity.gpu_step(ctx, s)
    ref = parity.oracle_step(cache, st, w, ref_inputs.to("cpu"), probe=so.out_token.cpu().numpy())
    parity.compare(mp, vo, so, ref, s.draft_len.cpu().numpy(), s.step,
                   s.seed.cpu().numpy().astype(np.uint64), bf16=True)
    ctx.close()


def test_zero_residual_mass_falls_back_to_p(cuda_device):
    V = 8
    ctx = od.Context(cuda_device, V, 7, 1, 1)
    vm = np.array([0, 1, 2, 3, 4, 5, 6, -1], np.int32)
    ctx.set_vocab_map(vm)
    ctx.cache_build(np.zeros((0, 4), np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32))
    dev = cuda_device
    logits = torch.zeros(1, 2, 8, dtype=torch.float32, device=dev)[:, :, :7]
    q_rows = torch.zeros(1, 1, 8, dtype=torch.float32, device=dev)
    q_rows[0, 0, :7] = 0.142857148
    d = torch.tensor([[7]], dtype=torch.int32, device=dev)
    klen = torch.tensor([1], dtype=torch.int32, device=dev)
    q_sel = torch.zeros(1, 1, dtype=torch.float32, device=dev)
    T = torch.ones(1, device=dev); seed = torch.zeros(1, dtype=torch.int64, device=dev)
    mp = od.od_map_proposals(ctx, d, klen, q_sel)
    vo = od.od_verify(ctx, logits, mp, T, seed, 0)
    so = od.od_sample_residual(ctx, logits, vo, q_rows, d, mp, T, seed, 0)
    torch.cuda.synchronize()
    assert int(mp.m[0]) == 0 and int(mp.tail_kind[0]) == od.OD_TAIL_UNMAPPED_STOP
    assert int(so.flags[0]) & od.OD_SF_ZERO_MASS
    cache = oracle.Cache(np.zeros((0, 4), np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32))
    ref = oracle.step_batch(cache, vm, 7, d.cpu().numpy(), klen.cpu().numpy(), q_sel.cpu().numpy(),
                            q_rows.cpu().numpy(), np.zeros((1, 2, 7), np.float32), oracle.DTYPE_F32,
                            np.ones(1, np.float32), np.zeros(1, np.uint64), 0)
    assert ref.flags[0] & oracle.FLAG_ZERO_MASS
    assert int(so.out_token[0]) == int(ref.token[0])
    assert float(so.resid_mass[0]) == pytest.approx(1.0, abs=1e-6)
    ctx.close()


def test_bad_temperature_and_invalid_ids_are_flagged_not_trapped(cuda_device):
    w = _small("badT", B=4, temperatures=(1.0, 0.7, 0.9, 0.5), gen_seed=0xBEEF80)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    s = synth.make_step(w, st, 0, device=cuda_device)
    s.temperature[1] = 0.0; s.temperature[2] = -1.0
    s.draft_ids[0, 0] = w.v_q + 5          # outside the draft vocabulary: treated as unmapped
    s.draft_ids[3, 0] = -3
    s.draft_len[:] = w.k_max
    st_ = parity.check_step(ctx, cache, st, w, s)
    mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
    torch.cuda.synchronize()
    assert int(mp.counters[od.OD_CNT_INVALID_IDS]) == 2
    ctx.close()


def test_lossless_on_the_gpu(cuda_device):
    """The GPU path itself keeps the target distribution: 8-token vocabulary,
    proposals drawn from q, 3 of 8 draft ids unmapped."""
    rng = np.random.default_rng(5)
    V, K, n = 8, 3, 60000
    vm = np.array([3, -1, 0, 7, -1, 5, -1, 2], np.int32)
    zq = rng.standard_normal((K, V)) * 1.5
    zq[:, vm < 0] += 1.0
    zp = (rng.standard_normal((K + 1, V)) * 1.5).astype(np.float32)
    q = torch.softmax(torch.from_numpy(zq), -1).float()
    ctx = od.Context(cuda_device, V, V, n, K)
    ctx.set_vocab_map(vm)
    ctx.cache_build(np.zeros((0, 4), np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32))
    dev = cuda_device
    g = torch.Generator(device="cpu"); g.manual_seed(1)
    counts = np.zeros(V)
    logits = torch.from_numpy(zp).to(dev).expand(n, K + 1, V).contiguous()
    q_rows = q.to(dev).expand(n, K, V).contiguous()
    for step in range(4):
        d = torch.stack([torch.multinomial(q[j], n, replacement=True, generator=g) for j in range(K)], 1)
        d = d.int().to(dev)
        q_sel = torch.gather(q_rows, 2, d.long().unsqueeze(-1)).squeeze(-1).contiguous()
        klen = torch.full((n,), K, dtype=torch.int32, device=dev)
        T = torch.ones(n, device=dev)
        seed = torch.arange(n, dtype=torch.int64, device=dev) + 77
        mp = od.od_map_proposals(ctx, d, klen, q_sel)
        vo = od.od_verify(ctx, logits, mp, T, seed, step)
        so = od.od_sample_residual(ctx, logits, vo, q_rows, d, mp, T, seed, step)
        torch.cuda.synchronize()
        nacc = vo.n_accepted.cpu().numpy()
        first = np.where(nacc > 0, mp.tgt_ids[:, 0].cpu().numpy(), so.out_token.cpu().numpy())
        counts += np.bincount(first, minlength=V)
    p0 = torch.softmax(torch.from_numpy(zp[0]).double(), -1).numpy()
    N = counts.sum()
    chi2 = ((counts - N * p0) ** 2 / (N * p0)).sum()
    assert chi2 < 7 + 5 * np.sqrt(14), (chi2, counts / N, p0)
    ctx.close()


# ------------------------------------------------------------ host-side validation
def test_argument_validation(cuda_device):
    L = od.lib()
    import ctypes as C
    with pytest.raises(od.OdError):
        od.Context(cuda_device, 100, 100, 4, 17)            # K_max beyond OD_MAX_K
    ctx = od.Context(cuda_device, 100, 120, 4, 4)
    dev = cuda_device
    d = torch.zeros(2, 4, dtype=torch.int32, device=dev)
    kl = torch.full((2,), 4, dtype=torch.int32, device=dev)
    qs = torch.full((2, 4), 0.1, device=dev)
    with pytest.raises(od.OdError) as e:                    # no vocabulary map yet
        od.od_map_proposals(ctx, d, kl, qs)
    assert e.value.status == -8
    bad = np.zeros(100, np.int32)                           # every id -> target 0
    with pytest.raises(od.OdError) as e:
        ctx.set_vocab_map(bad)
    assert e.value.status == -3
    too_big = np.arange(100, dtype=np.int32); too_big[5] = 120
    with pytest.raises(od.OdError) as e:
        ctx.set_vocab_map(too_big)
    assert e.value.status == -1
    ctx.set_vocab_map(np.arange(100, dtype=np.int32))
    with pytest.raises(od.OdError) as e:                    # n-gram longer than 4
        ctx.cache_build(np.array([[1, 2, 3, 4]], np.int32), np.array([5], np.int32), np.array([7], np.int32))
    assert e.value.status == -4
    with pytest.raises(od.OdError) as e:                    # id outside the draft vocabulary
        ctx.cache_build(np.array([[1, 200, -1, -1]], np.int32), np.array([2], np.int32), np.array([7], np.int32))
    assert e.value.status == -4
    ctx.cache_build(np.array([[1, 2, -1, -1]], np.int32), np.array([2], np.int32), np.array([110], np.int32))
    mp = od.od_map_proposals(ctx, d, kl, qs)
    T = torch.ones(2, device=dev); seed = torch.zeros(2, dtype=torch.int64, device=dev)
    store = torch.zeros(2 * 5 * 120 + 8, dtype=torch.bfloat16, device=dev)
    misaligned = store[1:1 + 2 * 5 * 120].view(2, 5, 120)   # base off by 2 bytes
    with pytest.raises(od.OdError) as e:
        od.od_verify(ctx, misaligned, mp, T, seed, 0)
    assert e.value.status == -2
    odd = torch.zeros(2, 5, 121, dtype=torch.bfloat16, device=dev)[:, :, :120]   # row stride 242 bytes
    with pytest.raises(od.OdError) as e:
        od.od_verify(ctx, odd, mp, T, seed, 0)
    assert e.value.status == -2
    with pytest.raises(od.OdError) as e:                    # batch beyond max_batch
        big = torch.zeros(5, 4, dtype=torch.int32, device=dev)
        od.od_map_proposals(ctx, big, torch.zeros(5, dtype=torch.int32, device=dev),
                            torch.zeros(5, 4, device=dev))
    assert e.value.status == -1
    with pytest.raises(TypeError):
        od.od_verify(ctx, torch.zeros(2, 5, 120, dtype=torch.float16, device=dev), mp, T, seed, 0)
    big_ctx = od.Context(cuda_device, 70000, 70000, 1, 2)   # draft ids do not fit a 16-bit key field
    big_ctx.set_vocab_map(np.arange(70000, dtype=np.int32))
    with pytest.raises(od.OdError) as e:
        big_ctx.cache_build(np.array([[1, 2, -1, -1]], np.int32), np.array([2], np.int32), np.array([7], np.int32))
    assert e.value.status == -5
    big_ctx.close()
    with pytest.raises(od.OdError) as e:                    # the sampler could not hold a row's tile values
        od.Context(cuda_device, 100, 7_000_000, 1, 2)
    assert e.value.status == -5
    torch.cuda.synchronize()
    ctx.close()


def test_host_step_matches_device_step(cuda_device):
    w = _small("host", B=12, v_q=2000, v_p=30000, cache_entries=500, gen_seed=0xBEEF90)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    ctx.host_step_reserve(od.OD_BF16)
    s = synth.make_step(w, st, 2, device=cuda_device)
    mp, vo, so = parity.gpu_step(ctx, s)
    h = s.to("cpu")
    pin = lambda t: t.contiguous().pin_memory()
    out = od.od_step_host(ctx, pin(h.draft_ids), pin(h.draft_len), pin(h.q_sel), pin(h.q_rows),
                          pin(h.logits), pin(h.temperature), pin(h.seed), s.step)
    assert torch.equal(out.n_accepted, vo.n_accepted.cpu())
    assert torch.equal(out.out_token, so.out_token.cpu())
    assert torch.equal(out.m, mp.m.cpu())
    assert torch.equal(out.n_draft_accepted, vo.n_draft_accepted.cpu())
    assert torch.equal(out.verify_flags, vo.flags.cpu())
    assert torch.equal(out.sample_flags, so.flags.cpu())
    ctx.close()


# ------------------------------------------------------------ adaptive drafting, exit rule
@pytest.mark.parametrize("gamma", [0.3, 0.7])
def test_exit_rule_matches_the_oracle(cuda_device, gamma):
    """Eq. (4)-(6): lengths equal the fp64 oracle's except where the kernel flagged a
    decision within its margin; probabilities within fp32 rounding."""
    from oracle import exit_rule as er
    rng = np.random.default_rng(11)
    B, K = 3000, 10
    f = rng.normal(2.0, 1.5, size=(B, K)).astype(np.float32)
    f[:50] = 40.0                                  # never exits
    f[50:100] = -40.0                              # exits at the first token
    avail = rng.integers(0, K + 1, size=B).astype(np.int32)
    ctx = od.Context(cuda_device, 100, 100, 4, K)
    length, reject, flags = od.od_exit_rule(ctx, torch.from_numpy(f).to(cuda_device),
                                            torch.from_numpy(avail).to(cuda_device), gamma)
    torch.cuda.synchronize()
    want_len, want_rej = er.exit_rule(f, avail, gamma)
    length, reject, flags = length.cpu().numpy(), reject.cpu().numpy(), flags.cpu().numpy()
    np.testing.assert_allclose(reject, want_rej, rtol=0, atol=3e-6)
    differ = length != want_len
    assert (flags[differ] != 0).all(), "a length that differs from the oracle's must be flagged"
    assert differ.sum() <= 3 and (flags != 0).sum() <= 10
    assert (length[avail == 0] == 0).all() and (length <= avail).all()
    # the result feeds od_map_proposals as draft_len: same dtype and shape
    assert length.dtype == np.int32 and length.shape == (B,)
    with pytest.raises(od.OdError):
        od.od_exit_rule(ctx, torch.zeros(2, K, device=cuda_device), None, 1.5)
    ctx.close()
