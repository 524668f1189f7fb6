"""Seeded random shapes through the whole step (and through the vocabulary-sharded step):
vocabulary sizes with ragged tails, every K_max, odd batch sizes, both logit types, dense
and sparse maps, with and without a cache; each compared with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_02659_b200 import binding as od
from paper_2507_02659_b200 import synth, vshard

import parity

pytestmark = pytest.mark.gpu


def _random_workload(rng, i):
    v_q = int(rng.integers(40, 3000))
    v_p = int(rng.integers(max(8, v_q // 2), 6000))
    k_max = int(rng.integers(1, od.OD_MAX_K + 1))
    kind = ["identity", "random"][int(rng.integers(0, 2))] if v_p >= v_q else "random"
    frac = float(rng.uniform(0.2, min(0.95, v_p / v_q * 0.9)))
    outside = v_p - (v_q if kind == "identity" else int(round(frac * v_q)))
    entries = int(rng.integers(0, 300)) if outside > 0 else 0
    return synth.Workload(
        f"fuzz{i}", B=int(rng.integers(1, 40)), steps=2, k_max=k_max, k_min=int(rng.integers(1, k_max + 1)),
        v_q=v_q, v_p=v_p, logit_dtype=["bf16", "f32"][int(rng.integers(0, 2))], map_kind=kind,
        mapped_frac=frac, cache_entries=entries, hit_prob=float(rng.uniform(0, 1)) if entries else 0.0,
        logit_kind=["corr", "noise", "zipf"][int(rng.integers(0, 3))], rho=0.9,
        temperatures=tuple(float(t) for t in rng.choice([0.3, 0.5, 0.7, 1.0, 1.5], size=3)),
        per_seq_seed=True, gen_seed=0xF00D00 + i, unmapped_shift=float(rng.uniform(0, 4)), sigma=2.0,
        # every third case: cached n-grams whose token collides with the direct map (the cases of
        # Eq. (2) overlap), made likely enough under the drafter to be rejected now and then
        targets_in_image=0.3 if i % 3 == 0 and entries else 0.0,
        targets_on_prefix=0.3 if i % 3 == 0 and entries else 0.0,
        plant_boost=8.0 if i % 3 == 0 and entries else 0.0)


@pytest.mark.parametrize("i", range(24))
def test_random_shapes_match_the_oracle(cuda_device, i):
    rng = np.random.default_rng(1000 + i)
    w = _random_workload(rng, i)
    st = synth.make_static(w)
    ctx = parity.make_context(w, st, cuda_device)
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    for step in range(2):
        s = synth.make_step(w, st, step, device=cuda_device)
        lg = parity.pad_rows(s.logits)
        parity.check_step(ctx, cache, st, w, s, logits=lg)
        # the same step with the vocabulary split into a random number of shards
        tiles = -(-w.v_p // 256)
        n = int(rng.integers(1, min(tiles, 6) + 1))
        mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
        vo, so, _ = vshard.emulate_step(ctx, lg, n, mp, s.q_rows, s.draft_ids, s.temperature, s.seed, s.step,
                                        copy_shards=bool(rng.integers(0, 2)))
        torch.cuda.synchronize()
        ref = parity.oracle_step(cache, st, w, s.to("cpu"), probe=so.out_token.cpu().numpy())
        parity.compare(mp, vo, so, ref, s.draft_len.cpu().numpy(), s.step,
                       s.seed.cpu().numpy().astype(np.uint64), bf16=(w.logit_dtype == "bf16"))
    ctx.close()
