"""Thin ctypes binding of libomnidraft.so (include/omnidraft.h).

Only argument marshalling lives here: tensors become raw device pointers, the
current torch stream becomes the `stream` argument, status codes become
exceptions. Every step of the path runs inside the CUDA library; there is no
CPU fallback: if the library is missing or a call fails, this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libomnidraft.so")

OD_F32, OD_BF16 = 0, 1
OD_ERR_INVALID_ARG, OD_ERR_ALIGNMENT = -1, -2
OD_TAIL_COMPLETE, OD_TAIL_UNMAPPED_STOP = 0, 1
OD_CNT_CACHE_HITS, OD_CNT_UNMAPPED_STOPS, OD_CNT_INVALID_IDS, OD_CNT_MAPPED_TOKENS = 0, 1, 2, 3
OD_CNT_COUNT = 4
OD_VF_BOUNDARY_MASK, OD_VF_BAD_TEMPERATURE, OD_VF_NONFINITE = 0xFFFF, 0x10000, 0x20000
OD_SF_BOUNDARY, OD_SF_ZERO_MASS, OD_SF_BAD_TEMPERATURE, OD_SF_BONUS = 0x1, 0x2, 0x4, 0x10
OD_TAU_ACCEPT, OD_TAU_SAMPLE, OD_TAU_EXIT = 1.0e-5, 2.0e-6, 4.0e-6
OD_MAX_K = 16
OD_NOALLOC_MAX_ROWS = 1024

EXPORTS = ["od_create", "od_destroy", "od_set_vocab_map", "od_cache_build", "od_set_option",
           "od_map_proposals", "od_verify", "od_sample_residual", "od_step", "od_host_step_reserve",
           "od_step_host", "od_verify_noalloc", "od_exit_rule", "od_cache_configure", "od_cache_set_clock",
           "od_cache_insert", "od_cache_trim", "od_cache_dump", "od_cache_stats", "od_distill_loss",
           "od_verify_shard_stats", "od_verify_shard_finish", "od_sample_shard_mass", "od_sample_shard_pick",
           "od_last_launch_info", "od_status_string", "od_version"]


class OdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().od_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


_lib = None


def lib():
    """The loaded library. Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2507_02659_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
        L.od_create.argtypes = [C.POINTER(vp), i32, i32, i32, i32, i32]
        L.od_destroy.argtypes = [vp]
        L.od_set_vocab_map.argtypes = [vp, vp]
        L.od_cache_build.argtypes = [vp, vp, vp, vp, i64]
        L.od_set_option.argtypes = [vp, C.c_char_p, i64]
        L.od_map_proposals.argtypes = [vp, i32, i32] + [vp] * 10 + [vp]
        L.od_verify.argtypes = [vp, i32, i32, vp, i32, i64, i64] + [vp] * 6 + [u64] + [vp] * 7 + [vp]
        L.od_sample_residual.argtypes = ([vp, i32, i32, vp, i32, i64, i64] + [vp] * 13 + [u64]
                                         + [vp] * 3 + [vp])
        L.od_step.argtypes = ([vp, i32, i32] + [vp] * 5 + [i32, i64, i64, vp, vp, u64] + [vp] * 17 + [vp])
        L.od_verify_noalloc.argtypes = [i32, i32, i32, vp, i32, i64, i64] + [vp] * 6 + [u64] + [vp] * 7 + [vp]
        L.od_exit_rule.argtypes = [vp, i32, i32, vp, vp, C.c_float, vp, vp, vp, vp]
        L.od_distill_loss.argtypes = ([vp, i32, i32] + [vp] * 7 + [i32, i64, i64] + [vp] * 4
                                      + [C.c_float, i32, vp, vp, vp])
        L.od_verify_shard_stats.argtypes = [vp, i32, i32, i32, i32, vp, i32, i64, i64] + [vp] * 4 + [vp]
        L.od_verify_shard_finish.argtypes = [vp, i32, i32, i32] + [vp] * 7 + [u64] + [vp] * 7 + [vp]
        L.od_sample_shard_mass.argtypes = [vp, i32, i32, i32, i32, vp, i32, i64, i64] + [vp] * 12 + [vp] + [vp]
        L.od_sample_shard_pick.argtypes = ([vp, i32, i32, i32, i32, i32, i32, vp, vp, i32, i64, i64] + [vp] * 13
                                           + [u64] + [vp] * 3 + [vp])
        L.od_cache_configure.argtypes = [vp, i64, i32, i32]
        L.od_cache_set_clock.argtypes = [vp, C.c_uint32]
        L.od_cache_insert.argtypes = [vp, i32, vp, vp, vp, vp]
        L.od_cache_trim.argtypes = [vp, vp]
        L.od_cache_dump.argtypes = [vp, i64, vp, vp, vp, vp, vp, C.POINTER(i64)]
        L.od_cache_stats.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)]
        L.od_host_step_reserve.argtypes = [vp, i32]
        L.od_step_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, i32, vp, vp, u64] + [vp] * 7 + [vp]
        L.od_last_launch_info.argtypes = [vp, i32]
        L.od_last_launch_info.restype = i64
        L.od_status_string.argtypes = [i32]
        L.od_status_string.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("od_status_string", "od_last_launch_info"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise OdError(status, where)


def _dp(t: Optional[torch.Tensor], dtype=None, device=None):
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    if device is not None and t.device != device:
        raise ValueError(f"tensor on {t.device}, context on {device}")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return C.c_void_p(t.data_ptr())


def _hp(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _stream(device) -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def logit_dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return OD_F32
    if t.dtype == torch.bfloat16:
        return OD_BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


class Context:
    """Owner of an od_ctx handle."""

    def __init__(self, device, draft_vocab: int, target_vocab: int, max_batch: int, max_k: int):
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise ValueError("a CUDA device is required")
        idx = self.device.index if self.device.index is not None else torch.cuda.current_device()
        self.device = torch.device("cuda", idx)
        torch.cuda.init()
        h = C.c_void_p()
        _check(lib().od_create(C.byref(h), idx, draft_vocab, target_vocab, max_batch, max_k), "od_create")
        self.handle = h
        self.draft_vocab, self.target_vocab = draft_vocab, target_vocab
        self.max_batch, self.max_k = max_batch, max_k

    def close(self):
        if getattr(self, "handle", None):
            lib().od_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_vocab_map(self, host_map):
        a = np.ascontiguousarray(host_map, dtype=np.int32)
        if a.shape != (self.draft_vocab,):
            raise ValueError("vocab map must have draft_vocab entries")
        _check(lib().od_set_vocab_map(self.handle, _hp(a)), "od_set_vocab_map")

    def cache_build(self, runs, run_len, run_target):
        runs = np.ascontiguousarray(runs, dtype=np.int32).reshape(-1, 4)
        run_len = np.ascontiguousarray(run_len, dtype=np.int32)
        run_target = np.ascontiguousarray(run_target, dtype=np.int32)
        E = int(run_len.shape[0])
        if runs.shape[0] != E or run_target.shape[0] != E:
            raise ValueError("cache arrays disagree on the number of entries")
        _check(lib().od_cache_build(self.handle, _hp(runs), _hp(run_len), _hp(run_target), E),
               "od_cache_build")

    # ---- online cache (insertion of unseen n-grams, LRU / LFU trim)
    def cache_configure(self, max_entries: int, policy: int, max_insert: int):
        _check(lib().od_cache_configure(self.handle, int(max_entries), int(policy), int(max_insert)),
               "od_cache_configure")

    def cache_set_clock(self, clock: int):
        _check(lib().od_cache_set_clock(self.handle, int(clock) & 0xFFFFFFFF), "od_cache_set_clock")

    def cache_insert(self, runs: torch.Tensor, run_len: torch.Tensor, run_target: torch.Tensor):
        d, i32 = self.device, torch.int32
        N = int(run_len.shape[0])
        if tuple(runs.shape) != (N, 4) or run_target.shape[0] != N:
            raise ValueError("candidates must be runs [N, 4], len [N], target [N]")
        _check(lib().od_cache_insert(self.handle, N, _dp(runs, i32, d), _dp(run_len, i32, d),
                                     _dp(run_target, i32, d), _stream(d)), "od_cache_insert")

    def cache_trim(self):
        _check(lib().od_cache_trim(self.handle, _stream(self.device)), "od_cache_trim")

    def cache_stats(self):
        """(entries, malformed candidates skipped, candidates lost to a full table) of the online cache."""
        e, i, d = C.c_int64(0), C.c_int64(0), C.c_int64(0)
        _check(lib().od_cache_stats(self.handle, C.byref(e), C.byref(i), C.byref(d)), "od_cache_stats")
        return e.value, i.value, d.value

    def cache_dump(self):
        """{run tuple: (target, last-access clock, frequency)} of the online cache (synchronous)."""
        n = C.c_int64(0)
        _check(lib().od_cache_dump(self.handle, 0, None, None, None, None, None, C.byref(n)), "od_cache_dump")
        E = n.value
        runs = np.full((max(E, 1), 4), -1, np.int32); ln = np.zeros(max(E, 1), np.int32)
        tg = np.zeros(max(E, 1), np.int32); st = np.zeros(max(E, 1), np.uint32); fr = np.zeros(max(E, 1), np.uint32)
        _check(lib().od_cache_dump(self.handle, E, _hp(runs), _hp(ln), _hp(tg), _hp(st), _hp(fr), C.byref(n)),
               "od_cache_dump")
        return {tuple(int(x) for x in runs[i, :ln[i]]): (int(tg[i]), int(st[i]), int(fr[i])) for i in range(E)}

    def set_option(self, name: str, value: int):
        _check(lib().od_set_option(self.handle, name.encode(), int(value)), "od_set_option")

    def last_launch_info(self, which: int) -> int:
        return int(lib().od_last_launch_info(self.handle, which))

    def host_step_reserve(self, logit_dtype: int):
        _check(lib().od_host_step_reserve(self.handle, logit_dtype), "od_host_step_reserve")


@dataclass
class MapOut:
    tgt_ids: torch.Tensor
    q_prime: torch.Tensor
    span_start: torch.Tensor
    span_len: torch.Tensor
    m: torch.Tensor
    tail_kind: torch.Tensor
    counters: torch.Tensor


@dataclass
class VerifyOut:
    row_max: torch.Tensor
    row_sum: torch.Tensor
    p_sel: torch.Tensor
    ratio: torch.Tensor
    n_accepted: torch.Tensor
    n_draft_accepted: torch.Tensor
    flags: torch.Tensor


@dataclass
class SampleOut:
    out_token: torch.Tensor
    resid_mass: torch.Tensor
    flags: torch.Tensor


def alloc_map_out(ctx: Context, B: int, K: int) -> MapOut:
    d = ctx.device
    z = lambda *s, dt=torch.int32: torch.zeros(*s, dtype=dt, device=d)
    return MapOut(z(B, K), z(B, K, dt=torch.float32), z(B, K), z(B, K), z(B),
                  z(B, dt=torch.uint8), z(OD_CNT_COUNT))


def alloc_verify_out(ctx: Context, B: int, K: int) -> VerifyOut:
    d = ctx.device
    f = lambda *s: torch.zeros(*s, dtype=torch.float32, device=d)
    i = lambda *s: torch.zeros(*s, dtype=torch.int32, device=d)
    return VerifyOut(f(B, K + 1), f(B, K + 1), f(B, K), f(B, K), i(B), i(B), i(B))


def alloc_sample_out(ctx: Context, B: int) -> SampleOut:
    d = ctx.device
    return SampleOut(torch.zeros(B, dtype=torch.int32, device=d),
                     torch.zeros(B, dtype=torch.float32, device=d),
                     torch.zeros(B, dtype=torch.int32, device=d))


def _strides(logits: torch.Tensor, B: int, K: int, v_p: int):
    if logits.dim() != 3 or logits.shape[0] != B or logits.shape[1] != K + 1 or logits.shape[2] != v_p:
        raise ValueError(f"logits must be [B, K+1, V_p], got {tuple(logits.shape)}")
    if logits.stride(2) != 1:
        raise ValueError("logit rows must be dense")
    return int(logits.stride(1)), int(logits.stride(0))


def od_map_proposals(ctx: Context, draft_ids, draft_len, q_sel, out: Optional[MapOut] = None) -> MapOut:
    B, K = draft_ids.shape
    out = out or alloc_map_out(ctx, B, K)
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    _check(lib().od_map_proposals(
        ctx.handle, B, K, _dp(draft_ids, i32, d), _dp(draft_len, i32, d), _dp(q_sel, f32, d),
        _dp(out.tgt_ids, i32, d), _dp(out.q_prime, f32, d), _dp(out.span_start, i32, d),
        _dp(out.span_len, i32, d), _dp(out.m, i32, d), _dp(out.tail_kind, torch.uint8, d),
        _dp(out.counters, i32, d), _stream(d)), "od_map_proposals")
    return out


def od_verify(ctx: Context, logits, mp: MapOut, temperature, seed, step: int,
              out: Optional[VerifyOut] = None) -> VerifyOut:
    B, K = mp.tgt_ids.shape
    out = out or alloc_verify_out(ctx, B, K)
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    rs, ss = _strides(logits, B, K, ctx.target_vocab)
    if logits.device != d:
        raise ValueError("logits on another device")
    _check(lib().od_verify(
        ctx.handle, B, K, C.c_void_p(logits.data_ptr()), logit_dtype_code(logits), rs, ss,
        _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        _dp(temperature, f32, d), _dp(seed, torch.int64, d), C.c_uint64(step & (2**64 - 1)),
        _dp(out.row_max, f32, d), _dp(out.row_sum, f32, d), _dp(out.p_sel, f32, d),
        _dp(out.ratio, f32, d), _dp(out.n_accepted, i32, d), _dp(out.n_draft_accepted, i32, d),
        _dp(out.flags, i32, d), _stream(d)), "od_verify")
    return out


def od_verify_noalloc(target_vocab: int, logits, mp: MapOut, temperature, seed, step: int,
                      out: VerifyOut) -> VerifyOut:
    """od_verify for callers that may not allocate device memory: no context, the
    kernels' scratch is a fixed array inside the library, and `out` must be passed
    in (this wrapper allocates nothing either). Works on the device of `logits`,
    which must be the current CUDA device."""
    B, K = mp.tgt_ids.shape
    d, i32, f32 = logits.device, torch.int32, torch.float32
    if d.type != "cuda" or d.index != torch.cuda.current_device():
        raise ValueError("logits must live on the current CUDA device")
    rs, ss = _strides(logits, B, K, target_vocab)
    _check(lib().od_verify_noalloc(
        target_vocab, B, K, C.c_void_p(logits.data_ptr()), logit_dtype_code(logits), rs, ss,
        _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        _dp(temperature, f32, d), _dp(seed, torch.int64, d), C.c_uint64(step & (2**64 - 1)),
        _dp(out.row_max, f32, d), _dp(out.row_sum, f32, d), _dp(out.p_sel, f32, d),
        _dp(out.ratio, f32, d), _dp(out.n_accepted, i32, d), _dp(out.n_draft_accepted, i32, d),
        _dp(out.flags, i32, d), _stream(d)), "od_verify_noalloc")
    return out


def od_distill_loss(ctx: Context, q_rows, draft_ids, mp: MapOut, logits, vo: VerifyOut, temperature,
                    lam: float, lambda_mode: int = 0, want_grad: bool = True, loss=None, grad=None):
    """Eq. (3) per draft position: (loss f32 [B, K], grad f32 [B, K, V_q] or None)."""
    B, K = mp.tgt_ids.shape
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    rs, ss = _strides(logits, B, K, ctx.target_vocab)
    if loss is None:
        loss = torch.zeros(B, K, dtype=f32, device=d)
    if grad is None and want_grad:
        grad = torch.empty(B, K, ctx.draft_vocab, dtype=f32, device=d)
    _check(lib().od_distill_loss(
        ctx.handle, B, K, _dp(q_rows, f32, d), _dp(draft_ids, i32, d), _dp(mp.tgt_ids, i32, d),
        _dp(mp.span_start, i32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        C.c_void_p(logits.data_ptr()), logit_dtype_code(logits), rs, ss, _dp(vo.row_max, f32, d),
        _dp(vo.row_sum, f32, d), _dp(vo.p_sel, f32, d), _dp(temperature, f32, d), C.c_float(lam),
        int(lambda_mode), _dp(loss, f32, d), _dp(grad, f32, d), _stream(d)), "od_distill_loss")
    return loss, grad


def od_exit_rule(ctx: Context, head_logits, avail_len, gamma: float):
    """Eq. (4)-(6): (draft_len int32 [B], reject_prob f32 [B, K], exit_flags int32 [B])."""
    B, K = head_logits.shape
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    draft_len = torch.zeros(B, dtype=i32, device=d)
    reject = torch.zeros(B, K, dtype=f32, device=d)
    flags = torch.zeros(B, dtype=i32, device=d)
    _check(lib().od_exit_rule(ctx.handle, B, K, _dp(head_logits, f32, d), _dp(avail_len, i32, d),
                              C.c_float(gamma), _dp(draft_len, i32, d), _dp(reject, f32, d),
                              _dp(flags, i32, d), _stream(d)), "od_exit_rule")
    return draft_len, reject, flags


def od_sample_residual(ctx: Context, logits, vo: VerifyOut, q_rows, draft_ids, mp: MapOut,
                       temperature, seed, step: int, out: Optional[SampleOut] = None) -> SampleOut:
    B, K = mp.tgt_ids.shape
    out = out or alloc_sample_out(ctx, B)
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    rs, ss = _strides(logits, B, K, ctx.target_vocab)
    if logits.device != d:
        raise ValueError("logits on another device")
    if tuple(q_rows.shape) != (B, K, ctx.draft_vocab):
        raise ValueError("q_rows must be [B, K, V_q]")
    _check(lib().od_sample_residual(
        ctx.handle, B, K, C.c_void_p(logits.data_ptr()), logit_dtype_code(logits), rs, ss,
        _dp(vo.row_max, f32, d), _dp(vo.row_sum, f32, d), _dp(q_rows, f32, d),
        _dp(draft_ids, i32, d), _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d),
        _dp(mp.span_start, i32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        _dp(mp.tail_kind, torch.uint8, d), _dp(vo.n_accepted, i32, d), _dp(temperature, f32, d),
        _dp(seed, torch.int64, d), C.c_uint64(step & (2**64 - 1)),
        _dp(out.out_token, i32, d), _dp(out.resid_mass, f32, d), _dp(out.flags, i32, d),
        _stream(d)), "od_sample_residual")
    return out


def od_step(ctx: Context, s_draft_ids, s_draft_len, s_q_sel, s_q_rows, logits, temperature, seed, step: int,
            mp: Optional[MapOut] = None, vo: Optional[VerifyOut] = None, so: Optional[SampleOut] = None):
    """Steps 1-3 in one call on device tensors: (MapOut, VerifyOut, SampleOut)."""
    B, K = s_draft_ids.shape
    mp = mp or alloc_map_out(ctx, B, K)
    vo = vo or alloc_verify_out(ctx, B, K)
    so = so or alloc_sample_out(ctx, B)
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    rs, ss = _strides(logits, B, K, ctx.target_vocab)
    if logits.device != d:
        raise ValueError("logits on another device")
    if tuple(s_q_rows.shape) != (B, K, ctx.draft_vocab):
        raise ValueError("q_rows must be [B, K, V_q]")
    _check(lib().od_step(
        ctx.handle, B, K, _dp(s_draft_ids, i32, d), _dp(s_draft_len, i32, d), _dp(s_q_sel, f32, d),
        _dp(s_q_rows, f32, d), C.c_void_p(logits.data_ptr()), logit_dtype_code(logits), rs, ss,
        _dp(temperature, f32, d), _dp(seed, torch.int64, d), C.c_uint64(step & (2**64 - 1)),
        _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d), _dp(mp.span_start, i32, d), _dp(mp.span_len, i32, d),
        _dp(mp.m, i32, d), _dp(mp.tail_kind, torch.uint8, d), _dp(mp.counters, i32, d),
        _dp(vo.row_max, f32, d), _dp(vo.row_sum, f32, d), _dp(vo.p_sel, f32, d), _dp(vo.ratio, f32, d),
        _dp(vo.n_accepted, i32, d), _dp(vo.n_draft_accepted, i32, d), _dp(vo.flags, i32, d),
        _dp(so.out_token, i32, d), _dp(so.resid_mass, f32, d), _dp(so.flags, i32, d), _stream(d)), "od_step")
    return mp, vo, so


# ---- the step with the target vocabulary split over GPUs (one call per phase) ----

def _shard_strides(logits: torch.Tensor, B: int, K: int, shard_len: int):
    if logits.dim() != 3 or logits.shape[0] != B or logits.shape[1] != K + 1 or logits.shape[2] != shard_len:
        raise ValueError(f"shard logits must be [B, K+1, shard_len], got {tuple(logits.shape)}")
    if logits.stride(2) != 1:
        raise ValueError("logit rows must be dense")
    return int(logits.stride(1)), int(logits.stride(0))


def od_verify_shard_stats(ctx: Context, shard_lo: int, logits, mp: MapOut, temperature,
                          out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Per-row records (c, s, M, x[t]) of this shard's columns: float32 [B, K+1, 4]."""
    B, K = mp.tgt_ids.shape
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    shard_len = int(logits.shape[2])
    rs, ss = _shard_strides(logits, B, K, shard_len)
    if out is None:
        out = torch.zeros(B, K + 1, 4, dtype=f32, device=d)
    _check(lib().od_verify_shard_stats(
        ctx.handle, B, K, shard_lo, shard_len, C.c_void_p(logits.data_ptr()), logit_dtype_code(logits),
        rs, ss, _dp(mp.tgt_ids, i32, d), _dp(mp.m, i32, d), _dp(temperature, f32, d), _dp(out, f32, d),
        _stream(d)), "od_verify_shard_stats")
    return out


def od_verify_shard_finish(ctx: Context, stats_all: torch.Tensor, mp: MapOut, temperature, seed, step: int,
                           out: Optional[VerifyOut] = None) -> VerifyOut:
    """stats_all: float32 [n_shards, B, K+1, 4], shard order."""
    B, K = mp.tgt_ids.shape
    if stats_all.dim() != 4 or tuple(stats_all.shape[1:]) != (B, K + 1, 4):
        raise ValueError("stats_all must be [n_shards, B, K+1, 4]")
    out = out or alloc_verify_out(ctx, B, K)
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    _check(lib().od_verify_shard_finish(
        ctx.handle, B, K, int(stats_all.shape[0]), _dp(stats_all, f32, d),
        _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        _dp(temperature, f32, d), _dp(seed, torch.int64, d), C.c_uint64(step & (2**64 - 1)),
        _dp(out.row_max, f32, d), _dp(out.row_sum, f32, d), _dp(out.p_sel, f32, d),
        _dp(out.ratio, f32, d), _dp(out.n_accepted, i32, d), _dp(out.n_draft_accepted, i32, d),
        _dp(out.flags, i32, d), _stream(d)), "od_verify_shard_finish")
    return out


def od_sample_shard_mass(ctx: Context, shard_lo: int, logits, vo: VerifyOut, q_rows, draft_ids, mp: MapOut,
                         temperature, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """This shard's shares of the sampling mass: float64 [B, 2]."""
    B, K = mp.tgt_ids.shape
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    shard_len = int(logits.shape[2])
    rs, ss = _shard_strides(logits, B, K, shard_len)
    if tuple(q_rows.shape) != (B, K, ctx.draft_vocab):
        raise ValueError("q_rows must be [B, K, V_q]")
    if out is None:
        out = torch.zeros(B, 2, dtype=torch.float64, device=d)
    _check(lib().od_sample_shard_mass(
        ctx.handle, B, K, shard_lo, shard_len, C.c_void_p(logits.data_ptr()), logit_dtype_code(logits),
        rs, ss, _dp(vo.row_max, f32, d), _dp(vo.row_sum, f32, d), _dp(q_rows, f32, d),
        _dp(draft_ids, i32, d), _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d),
        _dp(mp.span_start, i32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        _dp(mp.tail_kind, torch.uint8, d), _dp(vo.n_accepted, i32, d), _dp(temperature, f32, d),
        _dp(out, torch.float64, d), _stream(d)), "od_sample_shard_mass")
    return out


def od_sample_shard_pick(ctx: Context, shard_index: int, shard_lo: int, mass_all: torch.Tensor, logits,
                         vo: VerifyOut, q_rows, draft_ids, mp: MapOut, temperature, seed, step: int,
                         out: Optional[SampleOut] = None) -> SampleOut:
    """mass_all: float64 [n_shards, B, 2], shard order. Only the shard that holds the
    token writes it; the others write (-1, 0, 0)."""
    B, K = mp.tgt_ids.shape
    if mass_all.dim() != 3 or tuple(mass_all.shape[1:]) != (B, 2):
        raise ValueError("mass_all must be [n_shards, B, 2]")
    out = out or alloc_sample_out(ctx, B)
    d, i32, f32 = ctx.device, torch.int32, torch.float32
    shard_len = int(logits.shape[2])
    rs, ss = _shard_strides(logits, B, K, shard_len)
    _check(lib().od_sample_shard_pick(
        ctx.handle, B, K, int(mass_all.shape[0]), shard_index, shard_lo, shard_len,
        _dp(mass_all, torch.float64, d), C.c_void_p(logits.data_ptr()), logit_dtype_code(logits), rs, ss,
        _dp(vo.row_max, f32, d), _dp(vo.row_sum, f32, d), _dp(q_rows, f32, d),
        _dp(draft_ids, i32, d), _dp(mp.tgt_ids, i32, d), _dp(mp.q_prime, f32, d),
        _dp(mp.span_start, i32, d), _dp(mp.span_len, i32, d), _dp(mp.m, i32, d),
        _dp(mp.tail_kind, torch.uint8, d), _dp(vo.n_accepted, i32, d), _dp(temperature, f32, d),
        _dp(seed, torch.int64, d), C.c_uint64(step & (2**64 - 1)),
        _dp(out.out_token, i32, d), _dp(out.resid_mass, f32, d), _dp(out.flags, i32, d),
        _stream(d)), "od_sample_shard_pick")
    return out


@dataclass
class HostStepOut:
    n_accepted: torch.Tensor
    n_draft_accepted: torch.Tensor
    out_token: torch.Tensor
    tgt_ids: torch.Tensor
    m: torch.Tensor
    verify_flags: torch.Tensor
    sample_flags: torch.Tensor


def alloc_host_step_out(B: int, K: int, pin: bool = True) -> HostStepOut:
    z = lambda *s: torch.zeros(*s, dtype=torch.int32, pin_memory=pin)
    return HostStepOut(z(B), z(B), z(B), z(B, K), z(B), z(B), z(B))


def od_step_host(ctx: Context, draft_ids, draft_len, q_sel, q_rows, logits, temperature, seed,
                 step: int, out: Optional[HostStepOut] = None) -> HostStepOut:
    """Steps 1-3 on HOST tensors (pinned recommended); copies are part of the call."""
    B, K = draft_ids.shape
    out = out or alloc_host_step_out(B, K)
    cpu = torch.device("cpu")
    i32, f32 = torch.int32, torch.float32
    if tuple(logits.shape) != (B, K + 1, ctx.target_vocab) or not logits.is_contiguous():
        raise ValueError("logits must be a dense [B, K+1, V_p] host tensor")
    if logits.device != cpu:
        raise ValueError("od_step_host takes host tensors")
    _check(lib().od_step_host(
        ctx.handle, B, K, _dp(draft_ids, i32, cpu), _dp(draft_len, i32, cpu), _dp(q_sel, f32, cpu),
        _dp(q_rows, f32, cpu), C.c_void_p(logits.data_ptr()), logit_dtype_code(logits),
        _dp(temperature, f32, cpu), _dp(seed, torch.int64, cpu), C.c_uint64(step & (2**64 - 1)),
        _dp(out.n_accepted, i32, cpu), _dp(out.n_draft_accepted, i32, cpu), _dp(out.out_token, i32, cpu),
        _dp(out.tgt_ids, i32, cpu), _dp(out.m, i32, cpu), _dp(out.verify_flags, i32, cpu),
        _dp(out.sample_flags, i32, cpu), _stream(ctx.device)), "od_step_host")
    return out
