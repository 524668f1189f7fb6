"""The input generator: shapes, determinism, and the structure the workloads promise."""
import numpy as np
import torch

from paper_2507_02659_b200 import synth


def test_paper_configs_have_the_published_shapes():
    shapes = [(1, 4, 32000, "f32", 0), (1, 8, 128256, "bf16", 4096), (1, 10, 152064, "bf16", 65536),
              (64, 6, 128256, "bf16", 262144), (512, 8, 152064, "bf16", 262144)]
    for i, (B, K, vp, dt, E) in enumerate(shapes, start=1):
        w = synth.paper_config(i)
        assert (w.B, w.k_max, w.v_q, w.v_p, w.logit_dtype, w.cache_entries) == (B, K, 32000, vp, dt, E)
    w = synth.paper_config(6)      # same vocabulary on both sides: identity map, no cache
    assert (w.B, w.k_min, w.k_max, w.v_q, w.v_p, w.map_kind, w.cache_entries) == (256, 1, 8, 32000, 32000, "identity", 0)


def test_static_is_deterministic_and_well_formed():
    w = synth.scaled(synth.paper_config(2), v_q=500, v_p=900, cache_entries=200)
    a, b = synth.make_static(w), synth.make_static(w)
    np.testing.assert_array_equal(a.vocab_map, b.vocab_map)
    np.testing.assert_array_equal(a.runs, b.runs)
    mapped = a.vocab_map[a.vocab_map >= 0]
    assert mapped.size == 350 and np.unique(mapped).size == mapped.size
    assert ((a.run_len >= 2) & (a.run_len <= 4)).all()
    keys = {tuple(r[:l]) for r, l in zip(a.runs, a.run_len)}
    assert len(keys) == 200
    assert not np.isin(a.run_target, mapped).any()


def test_step_is_deterministic_and_consistent():
    w = synth.scaled(synth.paper_config(4), B=5, v_q=400, v_p=700, cache_entries=50, hit_prob=1.0)
    st = synth.make_static(w)
    s1, s2 = synth.make_step(w, st, 3), synth.make_step(w, st, 3)
    for f in ("draft_ids", "draft_len", "q_sel", "q_rows", "logits", "temperature", "seed"):
        assert torch.equal(getattr(s1, f), getattr(s2, f))
    assert s1.logits.dtype == torch.bfloat16 and tuple(s1.logits.shape) == (5, 7, 700)
    assert torch.allclose(s1.q_rows.sum(-1), torch.ones(5, 6), atol=1e-5)
    g = torch.gather(s1.q_rows, 2, s1.draft_ids.long().unsqueeze(-1)).squeeze(-1)
    assert torch.equal(g, s1.q_sel)
    assert ((s1.draft_len >= 1) & (s1.draft_len <= 6)).all()
    assert s1.seed.tolist() == [0, 1, 2, 3, 4]
    s3 = synth.make_step(w, st, 4)
    assert not torch.equal(s1.draft_ids, s3.draft_ids)
