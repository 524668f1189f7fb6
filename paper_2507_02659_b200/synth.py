"""Seeded synthetic inputs for the cross-vocabulary verification step.

This module only *makes inputs*: draft distributions, proposals, a vocabulary
map, an n-gram cache and target logits with the shapes of the paper's
draft/target pairs (Llama-68M's 32000-token vocabulary against 32000-,
128256- and 152064-token target vocabularies, App. A model table).  It holds
none of the method's arithmetic (no merge scan, no acceptance test, no
residual) and is imported by neither the CUDA library nor the CPU oracle: the
tests and the benchmark call it and hand the same bytes to both sides.

Everything is plain torch ops driven by one `torch.Generator`, so a step can be
produced on the CPU (small test shapes) or directly on the GPU (the batched
workloads, whose logits run to gigabytes).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np
import torch

N_MAX = 4  # longest cached run (draft tokens that merge into one target token)


@dataclass(frozen=True)
class Workload:
    name: str
    B: int                      # sequences per step
    steps: int                  # verification steps of the full workload
    k_max: int                  # draft tokens per step (upper bound)
    k_min: int                  # == k_max: fixed length; < k_max: K_b ~ U{k_min..k_max}
    v_q: int                    # draft vocabulary
    v_p: int                    # target vocabulary
    logit_dtype: str            # "f32" | "bf16"
    map_kind: str               # "identity" | "random"
    mapped_frac: float          # share of draft ids with a direct map ("random")
    cache_entries: int
    hit_prob: float             # chance that a sequence-step carries one planted cached run
    logit_kind: str             # "noise" | "zipf" | "corr"
    rho: float                  # correlation of target with mapped draft logits ("corr")
    temperatures: Tuple[float, ...]   # T_b = temperatures[b % len]
    per_seq_seed: bool          # verification seed_b = b, else 0
    gen_seed: int               # seed of the generator stream
    unmapped_shift: float = 4.0  # draft-logit penalty on ids with no direct map
    sigma: float = 3.0
    # Cache targets normally lie outside the map's image (a token whose text is one draft
    # token does not come back as a run). These shares put some inside it, to exercise the
    # collisions between the cases of Eq. (2):
    targets_in_image: float = 0.0    # share of entries whose target has a direct pre-image
    targets_on_prefix: float = 0.0   # share whose target is the image of the run's first id
    # Added to the draft logits of a planted run's ids, so that the drafter itself finds the run
    # likely (q' of the merged token is then large enough for the token to be rejected sometimes):
    plant_boost: float = 0.0


def paper_config(i: int) -> Workload:
    """The five workloads of the benchmark definition (1-based), and as number 6
    the same-vocabulary setting of the paper's Vicuna-7B experiments (Section 4.2:
    Llama-68M drafting for a target that shares its 32000-id tokenizer, so the map
    is the identity and the n-gram cache stays empty) as a larger ragged batch."""
    base = dict(v_q=32000, mapped_frac=0.7, sigma=3.0)
    if i == 1:
        return Workload("cfg1", B=1, steps=1000, k_max=4, k_min=4, v_p=32000,
                        logit_dtype="f32", map_kind="identity", cache_entries=0,
                        hit_prob=0.0, logit_kind="noise", rho=0.0,
                        temperatures=(1.0,), per_seq_seed=False,
                        gen_seed=0xDA7A0001, **base)
    if i == 2:
        return Workload("cfg2", B=1, steps=2000, k_max=8, k_min=8, v_p=128256,
                        logit_dtype="bf16", map_kind="random", cache_entries=4096,
                        hit_prob=0.2, logit_kind="zipf", rho=0.0,
                        temperatures=(1.0,), per_seq_seed=False,
                        gen_seed=0xDA7A0002, **base)
    if i == 3:
        return Workload("cfg3", B=1, steps=2000, k_max=10, k_min=1, v_p=152064,
                        logit_dtype="bf16", map_kind="random", cache_entries=65536,
                        hit_prob=0.2, logit_kind="corr", rho=0.8,
                        temperatures=(0.7,), per_seq_seed=False,
                        gen_seed=0xDA7A0003, **base)
    if i == 4:
        return Workload("cfg4", B=64, steps=500, k_max=6, k_min=1, v_p=128256,
                        logit_dtype="bf16", map_kind="random", cache_entries=262144,
                        hit_prob=0.2, logit_kind="corr", rho=0.8,
                        temperatures=(0.5, 0.7, 1.0), per_seq_seed=True,
                        gen_seed=0xDA7A0004, **base)
    if i == 5:
        return Workload("cfg5", B=512, steps=200, k_max=8, k_min=8, v_p=152064,
                        logit_dtype="bf16", map_kind="random", cache_entries=262144,
                        hit_prob=0.2, logit_kind="corr", rho=0.6,
                        temperatures=(1.0,), per_seq_seed=True,
                        gen_seed=0xDA7A0005, **base)
    if i == 6:
        return Workload("cfg6", B=256, steps=200, k_max=8, k_min=1, v_p=32000,
                        logit_dtype="bf16", map_kind="identity", cache_entries=0,
                        hit_prob=0.0, logit_kind="noise", rho=0.0,
                        temperatures=(0.7, 1.0), per_seq_seed=True,
                        gen_seed=0xDA7A0006, **base)
    raise ValueError(f"no such config: {i}")


def scaled(w: Workload, **kw) -> Workload:
    """A copy of `w` with some fields replaced (smaller B, vocabularies, ...)."""
    return replace(w, **kw)


@dataclass
class Static:
    """What does not change between steps: the map and the cache (host arrays)."""
    vocab_map: np.ndarray       # int32 [v_q], -1 = no direct map
    runs: np.ndarray            # int32 [E, 4], unused slots = -1
    run_len: np.ndarray         # int32 [E], 2..4
    run_target: np.ndarray      # int32 [E]


@dataclass
class StepInputs:
    draft_ids: torch.Tensor     # int32 [B, k_max]
    draft_len: torch.Tensor     # int32 [B]
    q_sel: torch.Tensor         # f32   [B, k_max]   q_rows[b, j, draft_ids[b, j]]
    q_rows: torch.Tensor        # f32   [B, k_max, v_q]
    logits: torch.Tensor        # f32 | bf16 [B, k_max + 1, v_p]
    temperature: torch.Tensor   # f32   [B]
    seed: torch.Tensor          # int64 [B] (the bit pattern of a uint64)
    step: int

    def to(self, device) -> "StepInputs":
        f = lambda t: t.to(device)
        return StepInputs(f(self.draft_ids), f(self.draft_len), f(self.q_sel),
                          f(self.q_rows), f(self.logits), f(self.temperature),
                          f(self.seed), self.step)

    def slice(self, lo: int, hi: int) -> "StepInputs":
        s = slice(lo, hi)
        return StepInputs(self.draft_ids[s], self.draft_len[s], self.q_sel[s],
                          self.q_rows[s], self.logits[s], self.temperature[s],
                          self.seed[s], self.step)


def make_static(w: Workload) -> Static:
    """Vocabulary map and n-gram cache contents, on the host, from `gen_seed`."""
    rng = np.random.default_rng(w.gen_seed)
    if w.map_kind == "identity":
        if w.v_p < w.v_q:
            raise ValueError("identity map needs v_p >= v_q")
        vocab_map = np.arange(w.v_q, dtype=np.int32)
    elif w.map_kind == "random":
        n_mapped = int(round(w.mapped_frac * w.v_q))
        if n_mapped > w.v_p:
            raise ValueError("more mapped ids than target ids")
        vocab_map = np.full(w.v_q, -1, dtype=np.int32)
        mapped_d = rng.permutation(w.v_q)[:n_mapped]
        mapped_t = rng.permutation(w.v_p)[:n_mapped]
        vocab_map[mapped_d] = mapped_t.astype(np.int32)
    else:
        raise ValueError(w.map_kind)

    E = w.cache_entries
    runs = np.full((E, N_MAX), -1, dtype=np.int32)
    run_len = np.zeros(E, dtype=np.int32)
    run_target = np.zeros(E, dtype=np.int32)
    if E > 0:
        in_image = np.zeros(w.v_p, dtype=bool)
        in_image[vocab_map[vocab_map >= 0]] = True
        outside = np.nonzero(~in_image)[0]
        if outside.size == 0:
            if w.targets_in_image + w.targets_on_prefix < 1.0:
                raise ValueError("cache targets need target ids outside the map's image")
            outside = np.arange(w.v_p)
        # distinct runs: draw, pack, de-duplicate, top up
        have = 0
        seen = set()
        while have < E:
            need = E - have
            ln = rng.integers(2, N_MAX + 1, size=need)
            ids = rng.integers(0, w.v_q, size=(need, N_MAX))
            for r in range(need):
                L = int(ln[r])
                key = tuple(int(x) for x in ids[r, :L])
                if key in seen:
                    continue
                seen.add(key)
                runs[have, :L] = ids[r, :L]
                run_len[have] = L
                have += 1
                if have == E:
                    break
        # several runs may share a target token: the cache can hold more
        # entries than there are target ids outside the image
        run_target[:] = outside[rng.integers(0, outside.size, size=E)]
        if w.targets_in_image > 0 or w.targets_on_prefix > 0:
            image = np.nonzero(in_image)[0]
            coin = rng.random(E)
            pick = image[rng.integers(0, max(1, image.size), size=E)] if image.size else run_target
            first = vocab_map[runs[:, 0]]
            on_prefix = (coin < w.targets_on_prefix) & (first >= 0)
            inside = ~on_prefix & (coin < w.targets_on_prefix + w.targets_in_image) & (image.size > 0)
            run_target[inside] = pick[inside]
            run_target[on_prefix] = first[on_prefix]
    return Static(vocab_map, runs, run_len, run_target)


def _torch_gen(w: Workload, step: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((w.gen_seed << 20) + step)
    return g


def make_step(w: Workload, st: Static, step: int, device="cpu",
              seq_chunk: int = 32) -> StepInputs:
    """Inputs of verification step `step` (deterministic in (w, step, device kind))."""
    dev = torch.device(device)
    g = _torch_gen(w, step, dev)
    B, K, Vq, Vp = w.B, w.k_max, w.v_q, w.v_p
    out_dtype = torch.float32 if w.logit_dtype == "f32" else torch.bfloat16

    temps = torch.tensor([w.temperatures[b % len(w.temperatures)] for b in range(B)],
                         dtype=torch.float32, device=dev)
    seeds = (torch.arange(B, dtype=torch.int64, device=dev) if w.per_seq_seed
             else torch.zeros(B, dtype=torch.int64, device=dev))
    vmap = torch.from_numpy(st.vocab_map).to(dev).long()
    mapped = vmap >= 0
    mapped_d = torch.nonzero(mapped).squeeze(1)
    mapped_t = vmap[mapped_d]

    # proposal lengths and planted runs are drawn on the host (tiny)
    hg = np.random.default_rng((w.gen_seed << 20) + step)
    if w.k_min == w.k_max:
        klen = np.full(B, K, dtype=np.int64)
    else:
        klen = hg.integers(w.k_min, K + 1, size=B)
    E = st.runs.shape[0]
    plant = np.full(B, -1, dtype=np.int64)      # entry planted in sequence b, or -1
    plant_off = np.zeros(B, dtype=np.int64)
    if E > 0 and w.hit_prob > 0:
        coin = hg.random(B) < w.hit_prob
        ent = hg.integers(0, E, size=B)
        offu = hg.random(B)
        for b in range(B):
            L = int(st.run_len[ent[b]])
            if coin[b] and L <= klen[b]:
                plant[b] = ent[b]
                plant_off[b] = int(offu[b] * (klen[b] - L + 1))

    draft_ids = torch.zeros(B, K, dtype=torch.int32, device=dev)
    q_sel = torch.zeros(B, K, dtype=torch.float32, device=dev)
    q_rows = torch.empty(B, K, Vq, dtype=torch.float32, device=dev)
    logits = torch.empty(B, K + 1, Vp, dtype=out_dtype, device=dev)

    shift = torch.zeros(Vq, dtype=torch.float32, device=dev)
    shift[~mapped] = w.unmapped_shift

    for lo in range(0, B, seq_chunk):
        hi = min(B, lo + seq_chunk)
        nb = hi - lo
        z_q = torch.randn(nb, K, Vq, generator=g, device=dev, dtype=torch.float32) * w.sigma
        T = temps[lo:hi].view(nb, 1, 1)
        if w.plant_boost > 0:
            for b in range(lo, hi):
                e = int(plant[b])
                for j in range(int(st.run_len[e]) if e >= 0 else 0):
                    z_q[b - lo, int(plant_off[b]) + j, int(st.runs[e, j])] += w.plant_boost
        qr = torch.softmax(((z_q - shift) / T).double(), dim=-1).float()
        q_rows[lo:hi] = qr
        ids = torch.multinomial(qr.view(nb * K, Vq), 1, generator=g).view(nb, K)
        # piece_start[b, i] = first draft position of the i-th proposed piece
        piece_start = torch.arange(K, device=dev).repeat(nb, 1)
        hit_row = torch.full((nb,), -1, dtype=torch.long, device=dev)
        hit_tok = torch.zeros(nb, dtype=torch.long, device=dev)
        for b in range(lo, hi):
            e = int(plant[b])
            if e < 0:
                continue
            L = int(st.run_len[e]); o = int(plant_off[b])
            ids[b - lo, o:o + L] = torch.from_numpy(st.runs[e, :L].astype(np.int64)).to(dev)
            ps = list(range(0, o + 1)) + list(range(o + L, K))
            ps = ps + [K - 1] * (K - len(ps))
            piece_start[b - lo] = torch.tensor(ps[:K], device=dev)
            hit_row[b - lo] = o
            hit_tok[b - lo] = int(st.run_target[e])
        draft_ids[lo:hi] = ids.int()
        q_sel[lo:hi] = torch.gather(qr, 2, ids.unsqueeze(-1)).squeeze(-1)

        # target logits, rows 0..K (row K has no draft row: fresh noise)
        noise = torch.randn(nb, K + 1, Vp, generator=g, device=dev, dtype=torch.float32)
        if w.logit_kind == "noise":
            # target = draft logits + N(0, 0.5^2) on the image of the map
            zp = noise * w.sigma
            src = z_q[:, :, mapped_d]
            zp[:, :K, mapped_t] = src + 0.5 * noise[:, :K, mapped_t]
        elif w.logit_kind == "zipf":
            zp = noise * w.sigma
            ntop = min(256, Vp)
            ranks = torch.arange(1, ntop + 1, device=dev, dtype=torch.float32)
            vals = 12.0 - 1.1 * torch.log(ranks)
            pick = torch.rand(nb, K + 1, Vp, generator=g, device=dev).topk(ntop, dim=-1).indices
            zp.scatter_(2, pick, vals.expand(nb, K + 1, ntop).contiguous())
        elif w.logit_kind == "corr":
            c = math.sqrt(max(0.0, 1.0 - w.rho * w.rho))
            zp = noise * w.sigma
            zq_piece = torch.gather(z_q, 1, piece_start.view(nb, K, 1).expand(nb, K, Vq))
            zp[:, :K, mapped_t] = w.rho * zq_piece[:, :, mapped_d] + c * zp[:, :K, mapped_t]
            for bb in range(nb):
                r = int(hit_row[bb])
                if r >= 0:
                    d1 = int(ids[bb, r])
                    tk = int(hit_tok[bb])
                    zp[bb, r, tk] = w.rho * z_q[bb, r, d1] + c * zp[bb, r, tk]
        else:
            raise ValueError(w.logit_kind)
        logits[lo:hi] = zp.to(out_dtype)
        del z_q, noise, zp, qr

    return StepInputs(draft_ids, torch.from_numpy(klen.astype(np.int32)).to(dev),
                      q_sel, q_rows, logits, temps, seeds, step)
