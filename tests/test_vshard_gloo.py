"""Vocabulary sharding, host side, with two CPU processes (gloo): the shard bounds
tile the vocabulary, the three exchanges deliver every rank's records in rank
order, and records merged across shards reproduce the statistics, the residual
mass and the token of the unsharded step. The oracle stands in for the GPU: a
rank's share of the residual mass is read off the oracle's CDF at the shard's
edges, its row records are plain sums over its own columns."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_02659_b200 import synth, vshard


def test_split_vocab_tiles_the_vocabulary():
    for v_p in (256, 1000, 32000, 128256, 152064):
        tiles = -(-v_p // 256)
        for world in (1, 2, 3, 8):
            if world > tiles:
                continue
            b = [vshard.split_vocab(v_p, r, world) for r in range(world)]
            assert b[0][0] == 0 and b[-1][1] == v_p
            for (lo, hi), (lo2, _) in zip(b, b[1:]):
                assert hi == lo2
            for lo, hi in b:
                assert lo % 256 == 0 and hi > lo and (hi % 256 == 0 or hi == v_p)
            n = [-(-(hi - lo) // 256) for lo, hi in b]
            assert max(n) - min(n) <= 1 and n == sorted(n, reverse=True)
    with pytest.raises(ValueError):
        vshard.split_vocab(500, 0, 3)          # two tiles cannot feed three shards
    with pytest.raises(ValueError):
        vshard.split_vocab(5000, 2, 2)


def test_combine_picks_takes_the_owner():
    tok = torch.tensor([[-1, 7, -1], [300, -1, -1], [-1, -1, -1]], dtype=torch.int32)
    mass = torch.tensor([[0.0, 0.25, 0.0], [0.5, 0.0, 0.0], [0.0, 0.0, 0.0]])
    fl = torch.tensor([[0, 1, 4], [0x10, 0, 4], [0, 0, 4]], dtype=torch.int32)
    t, m, f = vshard.combine_picks(tok, mass, fl)
    assert t.tolist() == [300, 7, -1] and m.tolist() == [0.5, 0.25, 0.0] and f.tolist() == [0x10, 1, 4]


def test_gather_shards_without_a_process_group_is_one_shard():
    x = torch.arange(6.0).view(2, 3)
    assert vshard.gather_shards(x).shape == (1, 2, 3)


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _worker(rank, world, port, out):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.scaled(synth.paper_config(4), B=9, v_q=600, v_p=1000, cache_entries=60,
                         hit_prob=0.7, rho=0.95)
        st = synth.make_static(w)
        s = synth.make_step(w, st, 3)
        cache = oracle.Cache(st.runs, st.run_len, st.run_target)
        lg, code = oracle.logits_to_numpy(s.logits)

        def run(probe=None):
            return oracle.step_batch(cache, st.vocab_map, w.v_p, s.draft_ids.numpy(), s.draft_len.numpy(),
                                     s.q_sel.numpy(), s.q_rows.numpy(), lg, code, s.temperature.numpy(),
                                     s.seed.numpy().astype(np.uint64), s.step, probe_token=probe, threads=1)
        full = run()
        B, K = w.B, w.k_max
        lo, hi = vshard.split_vocab(w.v_p, rank, world)
        x = s.logits.double().numpy()
        T = s.temperature.double().numpy()

        # exchange 1: row records of this rank's columns (maximum, sum relative to it, x[t_i])
        rec = np.zeros((B, K + 1, 4))
        for b in range(B):
            for r in range(int(full.m[b]) + 1):
                cols = x[b, r, lo:hi]
                M = cols.max()
                t = int(full.tgt_ids[b, r]) if r < full.m[b] else -1
                rec[b, r] = (M / T[b], np.exp((cols - M) / T[b]).sum(), M,
                             x[b, r, t] if lo <= t < hi else -np.inf)
        allrec = vshard.gather_shards(torch.from_numpy(rec)).numpy()
        assert allrec.shape == (world, B, K + 1, 4)
        np.testing.assert_array_equal(allrec[rank], rec)
        for b in range(B):
            for r in range(int(full.m[b]) + 1):
                M = allrec[:, b, r, 2].max()
                S = (allrec[:, b, r, 1] * np.exp((allrec[:, b, r, 2] - M) / T[b])).sum()
                assert M == full.row_max[b, r]
                assert abs(S / full.row_sum[b, r] - 1) < 1e-12
                if r < full.m[b]:
                    xt = allrec[:, b, r, 3].max()
                    assert abs(np.exp((xt - M) / T[b]) / S - full.p_sel[b, r]) < 1e-12

        # exchange 2: this rank's share of the mass = the oracle's CDF between the shard's edges
        before_lo = run(np.full(B, lo, np.int32)).probe_lo if lo > 0 else np.zeros(B)
        before_hi = run(np.full(B, hi, np.int32)).probe_lo if hi < w.v_p else full.mass.copy()
        share = torch.from_numpy(np.stack([before_hi - before_lo, np.zeros(B)], 1))
        mass_all = vshard.gather_shards(share).numpy()
        assert mass_all.shape == (world, B, 2)
        np.testing.assert_allclose(mass_all[:, :, 0].sum(0), full.mass, rtol=1e-12, atol=1e-15)

        # exchange 3: the shard in which u * R falls owns the token
        tok = np.full(B, -1, np.int32); msk = np.zeros(B, np.float32); fl = np.zeros(B, np.int32)
        ok = (full.flags & oracle.FLAG_ZERO_MASS) == 0
        for b in np.nonzero(ok)[0]:
            target = full.u_samp[b] * full.mass[b]
            cum = np.cumsum(mass_all[:, b, 0])
            owner = int(np.argmax(cum > target))
            if owner == rank:
                assert lo <= full.token[b] < hi
                tok[b] = full.token[b]; msk[b] = full.mass[b]; fl[b] = 0x10 if full.kind[b] == oracle.KIND_BONUS else 0
        pack = torch.stack([torch.from_numpy(tok), torch.from_numpy(msk).view(torch.int32), torch.from_numpy(fl)])
        allp = vshard.gather_shards(pack)
        t, mm, f = vshard.combine_picks(allp[:, 0], allp[:, 1].view(torch.float32), allp[:, 2])
        np.testing.assert_array_equal(t.numpy()[ok], full.token[ok])
        np.testing.assert_allclose(mm.numpy()[ok], full.mass[ok].astype(np.float32))
        assert ((f.numpy()[ok] == 0x10) == (full.kind[ok] == oracle.KIND_BONUS)).all()
        out.put((rank, "ok"))
    except Exception as e:  # pragma: no cover
        out.put((rank, repr(e)))
        raise
    finally:
        dist.destroy_process_group()


def test_two_rank_vocabulary_sharding_over_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
    res = sorted(out.get(timeout=5) for _ in range(2))
    assert res == [(0, "ok"), (1, "ok")], res
    assert all(p.exitcode == 0 for p in procs)
