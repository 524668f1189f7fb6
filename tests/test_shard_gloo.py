"""Batch sharding with two CPU processes (gloo): the slices cover the batch, the
gathered results are in sequence order, timings reduce to max / sum, and the
step on a slice equals the slice of the step on the whole batch (sequences are
independent), checked with the oracle standing in for the GPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_02659_b200 import shard, synth


def test_split_batch_covers_everything():
    for B in (0, 1, 7, 64, 511):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                lo, hi = shard.split_batch(B, r, world)
                assert 0 <= lo <= hi <= B
                got += list(range(lo, hi))
            assert got == list(range(B))
            sizes = [shard.split_batch(B, r, world) for r in range(world)]
            lens = [b - a for a, b in sizes]
            assert max(lens) - min(lens) <= 1
    with pytest.raises(ValueError):
        shard.split_batch(4, 2, 2)


def test_weak_shard_gives_each_rank_its_own_stream():
    w = synth.paper_config(4)
    a, b = shard.weak_shard(w, 0, 2), shard.weak_shard(w, 1, 2)
    assert a.B == b.B == w.B and a.gen_seed != b.gen_seed
    assert shard.weak_shard(w, 0, 1) is w


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _worker(rank, world, port, out):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.scaled(synth.paper_config(4), B=7, v_q=300, v_p=500, cache_entries=40,
                         hit_prob=0.7, rho=0.95)
        st = synth.make_static(w)
        s = synth.make_step(w, st, 5)
        cache = oracle.Cache(st.runs, st.run_len, st.run_target)

        def run(si):
            lg, code = oracle.logits_to_numpy(si.logits)
            return oracle.step_batch(cache, st.vocab_map, w.v_p, si.draft_ids.numpy(), si.draft_len.numpy(),
                                     si.q_sel.numpy(), si.q_rows.numpy(), lg, code, si.temperature.numpy(),
                                     si.seed.numpy().astype(np.uint64), si.step, threads=1)
        full = run(s)
        lo, hi = shard.split_batch(w.B, rank, world)
        mine = run(s.slice(lo, hi))
        np.testing.assert_array_equal(mine.n_accepted, full.n_accepted[lo:hi])
        np.testing.assert_array_equal(mine.token, full.token[lo:hi])
        n_all, t_all = shard.gather_step_results(torch.from_numpy(mine.n_accepted),
                                                 torch.from_numpy(mine.token), w.B)
        np.testing.assert_array_equal(n_all.numpy(), full.n_accepted)
        np.testing.assert_array_equal(t_all.numpy(), full.token)
        ms, units = shard.reduce_timing(10.0 + rank, 100 * (rank + 1), torch.device("cpu"))
        assert ms == 10.0 + world - 1 and units == 100 * world * (world + 1) // 2
        out.put((rank, "ok"))
    except Exception as e:  # pragma: no cover
        out.put((rank, repr(e)))
        raise
    finally:
        dist.destroy_process_group()


def test_two_rank_sharding_over_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
    res = sorted(out.get(timeout=5) for _ in range(2))
    assert res == [(0, "ok"), (1, "ok")], res
    assert all(p.exitcode == 0 for p in procs)
