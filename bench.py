#!/usr/bin/env python
"""Benchmark of the cross-vocabulary verification step (one JSON line).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..6] [--impl reference]

A step is one pass of the whole hot path (od_step: od_map_proposals -> od_verify
-> od_sample_residual) over one batch of synthetic input. The default workload
is the batched 128256-id configuration (config 4); steps cycle through a pool of
distinct input buffers larger than the L2 so every step's logits come from HBM.
The K timed steps are captured into one CUDA graph (the kernels run back to back
as in a decode loop) and timed with CUDA events between a barrier +
synchronize on both sides. The graph is then replayed for about 1.5 s, each
replay timed the same way, and `value` comes from the median replay: the
interval in which the clocks are sampled. With N > 1 every rank runs its own
full batch (weak scaling, no data-path collective) and the time is the max over
ranks; `--gpus N` without a torchrun environment starts the N ranks itself.

Also reported: `roofline` for od_verify (algorithmic logit bytes / its own
average launch duration from a graph of the same K launches, against the
measured HBM copy rate), `e2e` (the same metric through od_step_host with pinned
host buffers, copies inside the timed region), `cpu_baseline` (the CPU oracle as
it stands on a bounded sample), and the SM clocks seen during the timed region.

`--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "verified_draft_tokens_per_sec"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--pool", type=int, default=0, help="distinct step buffers (0 = enough for 4x L2)")
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--cache-update", action="store_true",
                    help="time the online-cache update path (insert + trim) instead of the verification step")
    ap.add_argument("--distill", action="store_true",
                    help="time the distillation loss + gradient (Eq. 3) of the step's proposals instead")
    ap.add_argument("--vocab-shards", type=int, default=0,
                    help="time one rank's kernels of the step with the target vocabulary split over this many GPUs")
    ap.add_argument("--shard-index", type=int, default=-1, help="the shard that is timed (default: the middle one)")
    ap.add_argument("--verify-grid", type=int, default=0, help="thread blocks of the streaming kernel (0 = one per multiprocessor)")
    ap.add_argument("--sample-tiles-per-warp", type=int, default=0)
    ap.add_argument("--no-pdl", action="store_true", help="plain stream-ordered launches")
    return ap.parse_args()


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        # nvidia-smi numbers the physical GPUs and ignores CUDA_VISIBLE_DEVICES: ask by UUID
        self.index = str(index)
        try:
            self.index = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
        except Exception:
            pass
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def ncu_traffic(workload: str):
    """Per-launch DRAM bytes (read + write) of the stream kernel from the committed ncu
    summary profiles/traffic.txt, or None when there is no figure for this workload or
    the kernel source has changed since the counters were taken. Line format:
    <workload> <bytes per launch> <sha256 of od_verify.cu at capture time>."""
    import hashlib
    try:
        src = os.path.join(ROOT, "paper_2507_02659_b200", "csrc", "od_verify.cu")
        with open(src, "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            for line in f:
                t = line.split()
                if len(t) >= 3 and not line.startswith("#") and t[0] == workload and t[2] == digest:
                    return float(t[1])
    except Exception:
        pass
    return None


def step_bytes(s):
    t = (s.draft_ids, s.draft_len, s.q_sel, s.q_rows, s.logits, s.temperature, s.seed)
    return sum(x.numel() * x.element_size() for x in t)


def host_step_bytes(s, w):
    """Bytes od_step_host copies to the device for step `s`: the small per-sequence arrays, and of
    the logits and the drafter's distributions only the rows the step can read (rows 0..K_b and
    0..K_b-1 of sequence b)."""
    small = sum(x.numel() * x.element_size() for x in (s.draft_ids, s.draft_len, s.q_sel, s.temperature, s.seed))
    kb = s.draft_len.clamp(0, w.k_max).long()
    rows_l = int((kb + 1).sum())
    rows_q = int(kb.sum())
    return small + rows_l * w.v_p * s.logits.element_size() + rows_q * w.v_q * 4


def oracle_time(w, st, host_steps, seconds):
    """Oracle on host cores over `host_steps` (CPU StepInputs, cycled), one full batch
    per step, until `seconds` have passed. Returns (tokens, elapsed_s, steps_done, threads)."""
    import oracle
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    threads = oracle.max_threads()
    prepared = []
    for s in host_steps:
        lg, code = oracle.logits_to_numpy(s.logits)
        prepared.append((s, (cache, st.vocab_map, w.v_p, s.draft_ids.numpy(), s.draft_len.numpy(),
                             s.q_sel.numpy(), s.q_rows.numpy(), lg, code, s.temperature.numpy(),
                             s.seed.numpy().astype(np.uint64))))
    tokens, elapsed, done = 0, 0.0, 0
    while elapsed < seconds:
        s, args = prepared[done % len(prepared)]
        t0 = time.perf_counter()
        oracle.step_batch(*args, done, threads=threads)
        elapsed += time.perf_counter() - t0
        tokens += int(s.draft_len.sum())
        done += 1
    return tokens, elapsed, done, threads


def run_reference(a):
    """The CPU oracle as the reference arm: rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2507_02659_b200 import synth
    w = synth.paper_config(a.config)
    st = synth.make_static(w)
    # one step = one full batch of the configuration
    sel = w.B
    w_s = w
    import oracle
    cache = oracle.Cache(st.runs, st.run_len, st.run_target)
    threads = oracle.max_threads()
    steps = []
    for i in range(a.warmup + a.steps):
        s = synth.make_step(w_s, st, i, device="cpu")
        lg, code = oracle.logits_to_numpy(s.logits)
        steps.append((s, lg, code))
        if len(steps) >= 8:
            break
    tokens, t_total = 0, 0.0
    for i in range(a.warmup + a.steps):
        s, lg, code = steps[i % len(steps)]
        t0 = time.perf_counter()
        oracle.step_batch(cache, st.vocab_map, w.v_p, s.draft_ids.numpy(), s.draft_len.numpy(),
                          s.q_sel.numpy(), s.q_rows.numpy(), lg, code, s.temperature.numpy(),
                          s.seed.numpy().astype(np.uint64), i, threads=threads)
        dt = time.perf_counter() - t0
        if i >= a.warmup:
            t_total += dt
            tokens += int(s.draft_len.sum())
    value = tokens / t_total
    sample = f"all {w.B} sequences of a step, {a.steps} steps (cycling {len(steps)} distinct steps)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": a.gpus,
        "steps": a.steps, "warmup": a.warmup, "ms_per_step": 1e3 * t_total / a.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "B": sel, "k_max": w.k_max,
                                         "draft_vocab": w.v_q, "target_vocab": w.v_p,
                                         "logit_dtype": w.logit_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_cache_update(a):
    """Online-cache maintenance (not part of the verification step): batches of 16384
    fresh candidates into a 262144-entry LRU cache, then the trim back to the bound.
    One JSON line: inserted candidates/s, and the trim against the bytes it must scan."""
    from paper_2507_02659_b200 import binding as od
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    v_q, v_p, bound, batch = 32000, 128256, 262144, 16384
    ctx = od.Context(dev, v_q, v_p, 4, 4)
    ctx.set_vocab_map(np.full(v_q, -1, np.int32))
    g = torch.Generator(device=dev); g.manual_seed(7)
    def cands():
        return (torch.randint(0, v_q, (batch, 4), generator=g, device=dev, dtype=torch.int32),
                torch.randint(2, 5, (batch,), generator=g, device=dev, dtype=torch.int32),
                torch.randint(0, v_p, (batch,), generator=g, device=dev, dtype=torch.int32))
    batches = [cands() for _ in range(20)]
    ins_ms, trim_ms = [], []
    # The calls are timed on the device, and the device must not wait for the host to submit
    # them (40 + 17 launches of a few microseconds each): a fill of 2 GiB goes in front of
    # each timed stretch, and the host queues the stretch while the device is busy with it.
    ballast = torch.empty(1 << 29, dtype=torch.float32, device=dev)
    for rep in range(max(3, a.warmup // 4) + 5):
        ctx.cache_configure(bound, 0, batch)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        torch.cuda.synchronize(dev)
        ballast.fill_(1.0)
        e[0].record()
        for t, (r, l, tg) in enumerate(batches):
            ctx.cache_set_clock(t + 1)
            ctx.cache_insert(r, l, tg)
        e[1].record()
        ballast.fill_(2.0)
        e[2].record()
        ctx.cache_trim()
        e[3].record()
        torch.cuda.synchronize(dev)
        ins_ms.append(e[0].elapsed_time(e[1])); trim_ms.append(e[2].elapsed_time(e[3]))
    ins, trim = statistics.median(ins_ms[3:]), statistics.median(trim_ms[3:])
    cap = 1 << 20                                             # slots: 2 x (bound + batch) rounded up
    live = bound + batch                                      # entries before the trim (an upper bound)
    # what a trim has to move: the table read once and the spare table cleared (24 bytes per
    # slot each), the live entries packed (32 bytes written, read again for the rebuild), the
    # survivors written (24 bytes); the select passes run over candidates only and add little
    scan_bytes = cap * 24 * 2 + live * 32 * 2 + bound * 24
    peak, peak_src = measured_peak()
    print(json.dumps({
        "metric": "cache_candidates_inserted_per_sec", "value": 20 * batch / (ins * 1e-3), "unit": "candidates/s",
        "n_gpus": 1, "higher_is_better": True, "dtype": "u64", "data": "synthetic",
        "config": {"workload": "online cache: 20 batches of 16384 candidates into a 262144-entry LRU cache, then trim"},
        "insert_us_per_batch": 1e3 * ins / 20, "trim_us": 1e3 * trim,
        "roofline": {"kernel": "od_cache_trim (pack live entries + clear, 13 radix-select passes over the "
                               "candidates, rebuild): 17 dependent launches, latency-bound", "bound": "hbm",
                     "achieved": scan_bytes / (trim * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": scan_bytes / (trim * 1e-3) / 1e9 / peak, "peak_source": peak_src,
                     "bytes_per_launch": scan_bytes, "traffic": None},
        "entries_after_trim": len(ctx.cache_dump())}))
    ctx.close()


def run_distill(a):
    """od_distill_loss on the bench workload's proposals (after od_map_proposals and
    od_verify, which are not timed): draft positions/s and the HBM rate of the drafter
    rows read and gradient rows written."""
    from paper_2507_02659_b200 import binding as od
    from paper_2507_02659_b200 import synth
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    w = synth.paper_config(a.config)
    st = synth.make_static(w)
    ctx = od.Context(dev, w.v_q, w.v_p, w.B, w.k_max)
    ctx.set_vocab_map(st.vocab_map)
    ctx.cache_build(st.runs, st.run_len, st.run_target)
    P = 6
    B, K = w.B, w.k_max
    pool = [synth.make_step(w, st, i, device=dev) for i in range(P)]
    mps = [od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel) for s in pool]
    vos = [od.od_verify(ctx, s.logits, mps[i], s.temperature, s.seed, i) for i, s in enumerate(pool)]
    loss = [torch.zeros(B, K, device=dev) for _ in range(P)]
    grad = [torch.empty(B, K, w.v_q, device=dev) for _ in range(P)]      # P x 49 MB: larger than L2 together with q
    def call(i):
        s = pool[i % P]
        od.od_distill_loss(ctx, s.q_rows, s.draft_ids, mps[i % P], s.logits, vos[i % P], s.temperature, 0.2, 0,
                           loss=loss[i % P], grad=grad[i % P])
    for i in range(max(3, a.warmup)):
        call(i)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(a.steps):
            call(i)
    g.replay(); torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); g.replay(); e1.record(); torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / a.steps
    active = sum(int(mps[i % P].span_len[torch.arange(K, device=dev)[None, :] < mps[i % P].m[:, None]].sum())
                 for i in range(a.steps)) / a.steps
    # active position: drafter row in, gradient row out, and (for the KL positions, nearly all) the target
    # row, whose gathered ids touch practically every 32-byte sector; other positions: zeros out
    esz_l = pool[0].logits.element_size()
    bytes_per_call = active * (2 * w.v_q * 4 + w.v_p * esz_l) + (B * K - active) * w.v_q * 4
    peak, peak_src = measured_peak()
    print(json.dumps({
        "metric": "distilled_draft_positions_per_sec", "value": active / (ms * 1e-3), "unit": "positions/s",
        "n_gpus": 1, "steps": a.steps, "warmup": a.warmup, "ms_per_step": ms, "higher_is_better": True,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "B": B, "k_max": K, "draft_vocab": w.v_q, "target_vocab": w.v_p,
                   "l2_policy": f"{P} distinct step buffers (q rows + gradient rows {P * 2 * B * K * w.v_q * 4 / 2**20:.0f} MiB)"},
        "roofline": {"kernel": "od_distill_kernel", "bound": "hbm", "achieved": bytes_per_call / (ms * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": bytes_per_call / (ms * 1e-3) / 1e9 / peak,
                     "peak_source": peak_src, "bytes_per_launch": bytes_per_call, "traffic": None},
        "active_positions_per_step": active}))
    ctx.close()


def run_vocab_shard(a):
    """One rank's share of a step whose target vocabulary is split over N GPUs: the
    five launches groups of that rank (od_map_proposals, od_verify_shard_stats,
    od_verify_shard_finish, od_sample_shard_mass, od_sample_shard_pick) on its own
    columns, timed on one GPU. The records of the other shards are computed
    beforehand and sit in the exchange buffers, so the decisions are those of the
    real step; the three all-gathers (16 B per row, 16 B and 12 B per sequence) are
    not part of the number."""
    from paper_2507_02659_b200 import binding as od
    from paper_2507_02659_b200 import synth, vshard
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    w = synth.paper_config(a.config)
    st = synth.make_static(w)
    N = a.vocab_shards
    r = a.shard_index if a.shard_index >= 0 else N // 2
    lo, hi = vshard.split_vocab(w.v_p, r, N)
    B, K = w.B, w.k_max
    ctx = od.Context(dev, w.v_q, w.v_p, B, K)
    ctx.set_vocab_map(st.vocab_map)
    ctx.cache_build(st.runs, st.run_len, st.run_target)
    full0 = synth.make_step(w, st, 0, device=dev)
    esz = full0.logits.element_size()
    shard_bytes = B * (K + 1) * (hi - lo) * esz
    P = max(3, -(-4 * L2_BYTES // shard_bytes))
    P = min(P, 64, a.steps + a.warmup)
    pool, shard_logits, mps, stats_all, mass_all, vos, sos = [], [], [], [], [], [], []
    for i in range(P):
        s = full0 if i == 0 else synth.make_step(w, st, i, device=dev)
        mp = od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel)
        bounds = [vshard.split_vocab(w.v_p, k, N) for k in range(N)]
        sa = torch.stack([od.od_verify_shard_stats(ctx, l, s.logits[:, :, l:h], mp, s.temperature) for l, h in bounds])
        vo = od.od_verify_shard_finish(ctx, sa, mp, s.temperature, s.seed, i)
        ma = torch.stack([od.od_sample_shard_mass(ctx, l, s.logits[:, :, l:h], vo, s.q_rows, s.draft_ids, mp,
                                                  s.temperature) for l, h in bounds])
        shard_logits.append(s.logits[:, :, lo:hi].contiguous())       # the rank's own dense buffer
        pool.append(synth.StepInputs(s.draft_ids, s.draft_len, s.q_sel, s.q_rows, shard_logits[-1],
                                     s.temperature, s.seed, s.step))
        mps.append(mp); stats_all.append(sa); mass_all.append(ma); vos.append(vo)
        sos.append(od.alloc_sample_out(ctx, B))
        del s
    torch.cuda.synchronize(dev)
    rows = [int((mps[i].m.clamp(0, K) + 1).sum().item()) for i in range(P)]
    toks = [int(pool[i].draft_len.sum().item()) for i in range(P)]

    def k1(i):
        s = pool[i]
        od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel, out=mps[i])

    def k2(i, step):
        s = pool[i]
        od.od_verify_shard_stats(ctx, lo, s.logits, mps[i], s.temperature, out=stats_all[i][r])
        od.od_verify_shard_finish(ctx, stats_all[i], mps[i], s.temperature, s.seed, i, out=vos[i])

    def k3(i, step):
        s = pool[i]
        od.od_sample_shard_mass(ctx, lo, s.logits, vos[i], s.q_rows, s.draft_ids, mps[i], s.temperature,
                                out=mass_all[i][r])
        od.od_sample_shard_pick(ctx, r, lo, mass_all[i], s.logits, vos[i], s.q_rows, s.draft_ids, mps[i],
                                s.temperature, s.seed, i, out=sos[i])

    def full_step(step):
        i = step % P
        k1(i); k2(i, step); k3(i, step)

    def graph_ms(fn):
        for step in range(max(3, a.warmup)):
            fn(step)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for step in range(a.steps):
                fn(a.warmup + step)
        g.replay(); torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); g.replay(); e1.record(); torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / a.steps

    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    ms_step = graph_ms(full_step)
    clocks = sampler.stop()
    ms_k2 = graph_ms(lambda step: k2(step % P, step))
    ms_k3 = graph_ms(lambda step: k3(step % P, step))
    row_bytes = (hi - lo) * esz
    k2_bytes = sum(rows[(a.warmup + k) % P] for k in range(a.steps)) / a.steps * row_bytes
    tokens = sum(toks[(a.warmup + k) % P] for k in range(a.steps)) / a.steps
    peak, peak_src = measured_peak()
    ach = k2_bytes / (ms_k2 * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": tokens / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": a.steps,
        "warmup": a.warmup, "ms_per_step": ms_step, "higher_is_better": True, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{w.name}, one of {N} vocabulary shards (shard {r}: target ids [{lo}, {hi}))",
                   "B": B, "k_max": K, "target_vocab": w.v_p, "logit_dtype": w.logit_dtype, "pool_buffers": P,
                   "l2_policy": f"{P} distinct shard buffers, {P * shard_bytes / 2**20:.0f} MiB of logits cycled",
                   "exchanges": "not timed: the other shards' records are precomputed in the exchange buffers"},
        "kernels_ms_per_step": {"od_verify_shard_stats+finish": ms_k2, "od_sample_shard_mass+pick": ms_k3},
        "roofline": {"kernel": "od_verify_shard_stats + od_verify_shard_finish", "bound": "hbm", "achieved": ach,
                     "peak": peak, "unit": "GB/s", "frac": ach / peak, "peak_source": peak_src,
                     "bytes_per_launch": k2_bytes, "traffic": None},
        "gpu_launches": 6 * a.steps, "clocks": clocks}))
    ctx.close()


def launcher_command(gpus: int, argv, port: int):
    """The command that starts `gpus` local ranks of this script (one per GPU) the way the
    scaling runs are started: torch.distributed.run on one node, rendezvous on 127.0.0.1."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def maybe_relaunch(a, argv, run=subprocess.call):
    """`--gpus N` (N > 1) outside a torchrun environment: start the N ranks and return their
    exit status; otherwise None (this process is a rank, or the only one)."""
    if a.gpus <= 1 or "WORLD_SIZE" in os.environ:
        return None
    return run(launcher_command(a.gpus, argv, free_port()))


def main():
    a = parse()
    rc = maybe_relaunch(a, sys.argv[1:])
    if rc is not None:
        sys.exit(rc)
    if a.impl == "reference":
        return run_reference(a)
    if a.distill:
        return run_distill(a)
    if a.cache_update:
        return run_cache_update(a)
    if a.vocab_shards:
        return run_vocab_shard(a)
    if a.warmup < 3:
        a.warmup = 3

    import torch.distributed as dist
    from paper_2507_02659_b200 import binding as od
    from paper_2507_02659_b200 import shard, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w0 = synth.paper_config(a.config)
    w = shard.weak_shard(w0, rank, world)
    st = synth.make_static(w)
    ctx = od.Context(dev, w.v_q, w.v_p, w.B, w.k_max)
    ctx.set_vocab_map(st.vocab_map)
    ctx.cache_build(st.runs, st.run_len, st.run_target)
    if a.verify_grid:
        ctx.set_option("verify_grid", a.verify_grid)
    # the pool's inputs are resident long before any timed launch: od_verify called on its own
    # (the roofline graph) may read rows 0, and the step's translation kernel the proposal,
    # before they wait for the launch in front
    ctx.set_option("early_inputs", 1)
    if a.sample_tiles_per_warp:
        ctx.set_option("sample_tiles_per_warp", a.sample_tiles_per_warp)
    if a.no_pdl:
        ctx.set_option("pdl", 0)

    # pool of distinct step buffers, > 4x L2 in logits so no step finds its rows in L2
    s0 = synth.make_step(w, st, 0, device=dev)
    logit_bytes = s0.logits.numel() * s0.logits.element_size()
    P = a.pool or max(3, -(-4 * L2_BYTES // logit_bytes))
    P = min(P, a.steps + a.warmup)
    pool = [s0] + [synth.make_step(w, st, i, device=dev) for i in range(1, P)]
    B, K = w.B, w.k_max
    esz = s0.logits.element_size()
    mps = [od.alloc_map_out(ctx, B, K) for _ in range(P)]
    vos = [od.alloc_verify_out(ctx, B, K) for _ in range(P)]
    sos = [od.alloc_sample_out(ctx, B) for _ in range(P)]

    def k1(i, step):
        s = pool[i]
        od.od_map_proposals(ctx, s.draft_ids, s.draft_len, s.q_sel, out=mps[i])

    def k2(i, step):
        s = pool[i]
        od.od_verify(ctx, s.logits, mps[i], s.temperature, s.seed, step, out=vos[i])

    def k3(i, step):
        s = pool[i]
        od.od_sample_residual(ctx, s.logits, vos[i], s.q_rows, s.draft_ids, mps[i], s.temperature,
                              s.seed, step, out=sos[i])

    def full_step(step):
        i = step % P
        s = pool[i]
        od.od_step(ctx, s.draft_ids, s.draft_len, s.q_sel, s.q_rows, s.logits, s.temperature, s.seed, step,
                   mp=mps[i], vo=vos[i], so=sos[i])

    # warm-up (also fills m for the K2-only graph)
    for step in range(a.warmup):
        full_step(step)
    for i in range(P):
        k1(i, 0)
    torch.cuda.synchronize(dev)
    rows_per_slot = [int((mps[i].m.clamp(0, K) + 1).sum().item()) for i in range(P)]
    tokens_per_slot = [int(pool[i].draft_len.sum().item()) for i in range(P)]

    def make_graph(fn, n, first):
        if a.no_graph:
            return None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for k in range(n):
                fn(first + k)
        return g

    g_step = make_graph(full_step, a.steps, a.warmup)
    g_k2 = make_graph(lambda step: k2(step % P, step), a.steps, a.warmup)
    g_k3 = make_graph(lambda step: k3(step % P, step), a.steps, a.warmup)
    g_k1 = make_graph(lambda step: k1(step % P, step), a.steps, a.warmup)

    def timed(g, fn):
        """ms for the K steps, device-timed between barrier + synchronize."""
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if g is not None:
            g.replay()
        else:
            for k in range(a.steps):
                fn(a.warmup + k)
        e1.record()
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        return e0.elapsed_time(e1)

    # one untimed replay of each graph, then the timed region
    for g in (g_step, g_k2, g_k3, g_k1):
        if g is not None:
            g.replay()
    torch.cuda.synchronize(dev)
    clocks = ClockSampler(local)
    if rank == 0:
        clocks.start()
        time.sleep(0.3)
    ms_first = timed(g_step, full_step)
    # The same K steps again and again for about 1.5 s, each replay timed like the first: the
    # clocks are sampled over this window, and the headline number is its median replay.
    extra, t_end = [ms_first], time.perf_counter() + 1.5
    while time.perf_counter() < t_end and len(extra) < 400:
        extra.append(timed(g_step, full_step))
    if world > 1:                                   # every rank must take the same number of replays
        n_rep = torch.tensor([len(extra)], device=dev)
        dist.all_reduce(n_rep, op=dist.ReduceOp.MIN)
        extra = extra[:int(n_rep.item())]
    ms_step = statistics.median(extra)
    ms_k2 = timed(g_k2, lambda step: k2(step % P, step))
    ms_k3 = timed(g_k3, lambda step: k3(step % P, step))
    ms_k1 = timed(g_k1, lambda step: k1(step % P, step))
    clk = clocks.stop() if rank == 0 else None

    steps_idx = [(a.warmup + k) % P for k in range(a.steps)]
    tokens_local = sum(tokens_per_slot[i] for i in steps_idx)
    rows_total = sum(rows_per_slot[i] for i in steps_idx)
    ms_max, tokens_all = shard.reduce_timing(ms_step, tokens_local, dev)
    value = tokens_all / (ms_max * 1e-3)

    k2_bytes_per_launch = rows_total * w.v_p * esz / a.steps
    k2_ms_per_launch = ms_k2 / a.steps
    achieved = k2_bytes_per_launch / (k2_ms_per_launch * 1e-3) / 1e9
    peak, peak_src = measured_peak()

    # end to end through od_step_host: pinned host inputs, copies inside the timed region
    e2e = None
    if not a.no_e2e:
        ctx.host_step_reserve(od.OD_BF16 if w.logit_dtype == "bf16" else od.OD_F32)
        hp = min(2, P)
        hosts = []
        for i in range(hp):
            h = pool[i].to("cpu")
            hosts.append(synth.StepInputs(*[t.contiguous().pin_memory() for t in
                                            (h.draft_ids, h.draft_len, h.q_sel, h.q_rows, h.logits,
                                             h.temperature, h.seed)], h.step))
        hout = od.alloc_host_step_out(B, K)
        n_e = max(1, a.e2e_steps)

        def host_step(k):
            h = hosts[k % hp]
            od.od_step_host(ctx, h.draft_ids, h.draft_len, h.q_sel, h.q_rows, h.logits, h.temperature,
                            h.seed, k, out=hout)
        for k in range(3):
            host_step(k)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(n_e):
            host_step(k)
        e1.record()
        torch.cuda.synchronize(dev)
        ms_e = e0.elapsed_time(e1)
        tok_e = sum(int(hosts[k % hp].draft_len.sum()) for k in range(n_e))
        ms_e_max, tok_e_all = shard.reduce_timing(ms_e, tok_e, dev)
        d2h = sum(t.numel() * t.element_size() for t in
                  (hout.n_accepted, hout.n_draft_accepted, hout.out_token, hout.tgt_ids, hout.m,
                   hout.verify_flags, hout.sample_flags))
        e2e = {"value": tok_e_all / (ms_e_max * 1e-3), "unit": UNIT, "steps": n_e,
               "ms_per_step": ms_e_max / n_e, "h2d_bytes_per_step": host_step_bytes(hosts[0], w),
               "d2h_bytes_per_step": d2h, "api": "od_step_host (pinned host buffers)"}

    cpu = None
    if rank == 0 and world == 1 and not a.no_cpu_baseline:
        nseq = min(w.B, 64)
        host_steps = [pool[i].slice(0, nseq).to("cpu") for i in range(min(P, 3))]
        tok, el, done, threads = oracle_time(w, st, host_steps, a.cpu_seconds)
        cpu = {"value": tok / el, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{done} steps of {nseq} of the batch's {w.B} sequences, cycling {len(host_steps)} "
                         f"distinct steps ({el:.1f} s of oracle time)"}

    if rank == 0:
        # what the timed steps decided (the pool slots hold the outputs of their last step)
        acc = sum(int(vos[i].n_accepted.sum().item()) for i in steps_idx)
        acc_draft = sum(int(vos[i].n_draft_accepted.sum().item()) for i in steps_idx)
        prop = sum(tokens_per_slot[i] for i in steps_idx)
        mapped = sum(int(mps[i].m.clamp(0, K).sum().item()) for i in steps_idx)
        vflag = sum(int((vos[i].flags & od.OD_VF_BOUNDARY_MASK != 0).sum().item()) for i in steps_idx)
        vbits = sum(int(sum(((vos[i].flags >> k) & 1).sum().item() for k in range(K))) for i in steps_idx)
        sflag = sum(int((sos[i].flags & od.OD_SF_BOUNDARY != 0).sum().item()) for i in steps_idx)
        bonus = sum(int((sos[i].flags & od.OD_SF_BONUS != 0).sum().item()) for i in steps_idx)
        zero = sum(int((sos[i].flags & od.OD_SF_ZERO_MASS != 0).sum().item()) for i in steps_idx)
        stops = sum(int((mps[i].tail_kind == od.OD_TAIL_UNMAPPED_STOP).sum().item()) for i in steps_idx)
        hits = sum(int((mps[i].span_len[torch.arange(K, device=dev)[None, :] < mps[i].m[:, None]] >= 2).sum().item())
                   for i in steps_idx)
        n_seq = B * a.steps
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": a.steps,
            "warmup": a.warmup, "ms_per_step": ms_max / a.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w0.name, "B_per_gpu": w.B, "k_max": w.k_max, "draft_vocab": w.v_q,
                       "target_vocab": w.v_p, "logit_dtype": w.logit_dtype,
                       "cache_entries": w.cache_entries, "pool_buffers": P,
                       "l2_policy": f"inputs larger than L2: {P} distinct step buffers, "
                                    f"{P * logit_bytes / 2**20:.0f} MiB of logits cycled",
                       "launch": ("K steps (one od_step call each) captured in one CUDA graph, replayed for 1.5 s; "
                                  "value from the median replay") if not a.no_graph else "eager launches",
                       "roofline_launch": "od_verify alone, K calls in one graph",
                       "options": "early_inputs = 1 for every launch (the pool's inputs are resident "
                                  "before any timed launch)",
                       "parallelism": f"batch sharding x{world}, no collective"},
            # od_step: translation, streaming pass, sampler (which takes step 2's decisions);
            # without programmatic dependent launch the decide kernel is a launch of its own
            "gpu_launches": (4 if a.no_pdl else 3) * a.steps,
            "kernels_ms_per_step": {"od_map_proposals": ms_k1 / a.steps, "od_verify": ms_k2 / a.steps,
                                    "od_sample_residual": ms_k3 / a.steps,
                                    "step_replays": len(extra),
                                    "first_replay_ms_per_step": ms_first / a.steps},
            "roofline": {"kernel": "od_verify (od_verify_stream_kernel + od_verify_decide_kernel)", "bound": "hbm", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                         "bytes_per_launch": k2_bytes_per_launch,
                         "us_per_launch": 1e3 * k2_ms_per_launch,
                         "frac_of_theoretical_8184": achieved / 8184.0,
                         "traffic": ncu_traffic(w0.name)},
            "e2e": e2e, "cpu_baseline": cpu, "clocks": clk,
            "stats": {"acceptance_rate": acc_draft / max(1, prop), "rows_per_step": rows_total / a.steps,
                      "draft_tokens_per_step": tokens_local / a.steps,
                      "mean_accepted_length": acc / n_seq,
                      "accepted_target_tokens_per_sec": (acc + n_seq) / (ms_max * 1e-3),
                      "mapped_target_tokens": mapped, "cache_hits": hits, "unmapped_stops": stops,
                      "accept_decisions": mapped, "accept_decisions_flagged": vbits,
                      "sequences_with_a_flagged_accept_decision": vflag,
                      "extra_tokens": n_seq, "extra_tokens_flagged": sflag, "free_tokens": bonus,
                      "zero_residual_mass": zero,
                      "verify_grid": ctx.last_launch_info(0), "verify_span_a": ctx.last_launch_info(1),
                      "sample_grid": ctx.last_launch_info(2)},
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
