"""ctypes front end of the CPU oracle (od_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It knows nothing about the CUDA library and the
CUDA library knows nothing about it.  All arithmetic lives in od_oracle.c; this
file only compiles it (gcc, -O2, OpenMP) and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "od_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

TAIL_COMPLETE, TAIL_UNMAPPED_STOP = 0, 1
KIND_RESIDUAL, KIND_BONUS = 0, 1
FLAG_ZERO_MASS, FLAG_BAD_TEMPERATURE = 1, 2
DTYPE_F32, DTYPE_BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile od_oracle.c into liboracle.so next to it (no-op when fresh)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".{os.getpid()}.tmp"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_uniform.restype = C.c_double
        _lib.oracle_uniform.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32]
        _lib.oracle_cache_create.restype = C.c_void_p
        _lib.oracle_cache_create.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64]
        _lib.oracle_cache_destroy.argtypes = [C.c_void_p]
        _lib.oracle_cache_size.restype = C.c_int64
        _lib.oracle_cache_size.argtypes = [C.c_void_p]
        _lib.oracle_cache_lookup.restype = C.c_int32
        _lib.oracle_cache_lookup.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        _lib.oracle_openmp_threads.restype = C.c_int32
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def uniform(seed: int, step: int, position: int, tag: int) -> float:
    return float(lib().oracle_uniform(seed & (2**64 - 1), step & (2**64 - 1), position, tag))


class Cache:
    """The n-gram cache C as an exact-match dictionary (Section 3.1)."""

    def __init__(self, runs, run_len, run_target):
        runs = np.ascontiguousarray(runs, dtype=np.int32).reshape(-1, 4)
        run_len = np.ascontiguousarray(run_len, dtype=np.int32)
        run_target = np.ascontiguousarray(run_target, dtype=np.int32)
        self._h = lib().oracle_cache_create(_p(runs), _p(run_len), _p(run_target),
                                            int(run_len.shape[0]))
        if not self._h:
            raise ValueError("malformed cache entry (run length must be 2..4)")

    def __len__(self):
        return int(lib().oracle_cache_size(self._h))

    def lookup(self, ids) -> int:
        a = np.ascontiguousarray(ids, dtype=np.int32)
        return int(lib().oracle_cache_lookup(self._h, _p(a), int(a.shape[0])))

    def __del__(self):
        try:
            if self._h:
                lib().oracle_cache_destroy(self._h)
                self._h = None
        except Exception:
            pass


@dataclass
class StepResult:
    tgt_ids: np.ndarray        # i32 [B,K]
    q_prime: np.ndarray        # f64 [B,K]
    span_start: np.ndarray     # i32 [B,K]
    span_len: np.ndarray       # i32 [B,K]
    m: np.ndarray              # i32 [B]
    tail_kind: np.ndarray      # i32 [B]
    hits: np.ndarray           # i32 [B]
    row_max: np.ndarray        # f64 [B,K+1]
    row_sum: np.ndarray        # f64 [B,K+1]
    p_sel: np.ndarray          # f64 [B,K]
    ratio: np.ndarray          # f64 [B,K]
    u_acc: np.ndarray          # f64 [B,K]
    accept: np.ndarray         # i32 [B,K]
    n_accepted: np.ndarray     # i32 [B]
    n_draft_accepted: np.ndarray  # i32 [B]
    kind: np.ndarray           # i32 [B]
    token: np.ndarray          # i32 [B]
    mass: np.ndarray           # f64 [B]
    u_samp: np.ndarray         # f64 [B]
    cdf_lo: np.ndarray         # f64 [B]  CDF interval of `token`
    cdf_hi: np.ndarray
    probe_lo: np.ndarray       # f64 [B]  CDF interval of the probed token
    probe_hi: np.ndarray
    flags: np.ndarray          # i32 [B]


def step_batch(cache: Cache, vocab_map, v_p: int, draft_ids, draft_len, q_sel,
               q_rows, logits, logit_dtype: int, temperature, seed, step: int,
               probe_token=None, threads: int = 0,
               row_stride: Optional[int] = None,
               seq_stride: Optional[int] = None) -> StepResult:
    """One verification step for B independent sequences.

    `logits` is a numpy array [B, K+1, v_p] of float32, or of uint16 holding
    bf16 bit patterns.  `seed` is uint64 [B].
    """
    vocab_map = np.ascontiguousarray(vocab_map, dtype=np.int32)
    draft_ids = np.ascontiguousarray(draft_ids, dtype=np.int32)
    B, K = draft_ids.shape
    draft_len = np.ascontiguousarray(draft_len, dtype=np.int32)
    q_sel = np.ascontiguousarray(q_sel, dtype=np.float32)
    q_rows = np.ascontiguousarray(q_rows, dtype=np.float32)
    v_q = int(vocab_map.shape[0])
    assert q_rows.shape == (B, K, v_q), q_rows.shape
    want = np.float32 if logit_dtype == DTYPE_F32 else np.uint16
    logits = np.ascontiguousarray(logits)
    assert logits.dtype == want, (logits.dtype, want)
    if row_stride is None:
        assert logits.shape == (B, K + 1, v_p), logits.shape
        row_stride, seq_stride = v_p, (K + 1) * v_p
    temperature = np.ascontiguousarray(temperature, dtype=np.float32)
    seed = np.ascontiguousarray(seed).astype(np.uint64)
    probe = None if probe_token is None else np.ascontiguousarray(probe_token, dtype=np.int32)
    if threads <= 0:
        threads = int(lib().oracle_openmp_threads())

    i32 = lambda *s: np.zeros(s, dtype=np.int32)
    f64 = lambda *s: np.zeros(s, dtype=np.float64)
    r = StepResult(i32(B, K), f64(B, K), i32(B, K), i32(B, K), i32(B), i32(B), i32(B),
                   f64(B, K + 1), f64(B, K + 1), f64(B, K), f64(B, K), f64(B, K),
                   i32(B, K), i32(B), i32(B), i32(B), i32(B), f64(B), f64(B), f64(B),
                   f64(B), f64(B), f64(B), i32(B))
    lib().oracle_step_batch(
        C.c_void_p(cache._h), _p(vocab_map), C.c_int32(v_q), C.c_int64(v_p),
        C.c_int32(B), C.c_int32(K), _p(draft_ids), _p(draft_len), _p(q_sel),
        _p(q_rows), _p(logits), C.c_int32(logit_dtype), C.c_int64(row_stride),
        C.c_int64(seq_stride), _p(temperature), _p(seed), C.c_uint64(step),
        _p(probe), C.c_int32(threads),
        _p(r.tgt_ids), _p(r.q_prime), _p(r.span_start), _p(r.span_len), _p(r.m),
        _p(r.tail_kind), _p(r.hits), _p(r.row_max), _p(r.row_sum), _p(r.p_sel),
        _p(r.ratio), _p(r.u_acc), _p(r.accept), _p(r.n_accepted),
        _p(r.n_draft_accepted), _p(r.kind), _p(r.token), _p(r.mass), _p(r.u_samp),
        _p(r.cdf_lo), _p(r.cdf_hi), _p(r.probe_lo), _p(r.probe_hi), _p(r.flags))
    return r


def map_sequence(cache: Cache, vocab_map, draft_ids, q_sel):
    """Eq. (1) for one proposal: (tgt, q_prime, span_start, span_len, m, tail, hits)."""
    vocab_map = np.ascontiguousarray(vocab_map, dtype=np.int32)
    d = np.ascontiguousarray(draft_ids, dtype=np.int32)
    K = int(d.shape[0])
    q = np.ascontiguousarray(q_sel, dtype=np.float32)
    tgt = np.zeros(max(K, 1), np.int32); qp = np.zeros(max(K, 1), np.float64)
    ss = np.zeros(K + 1, np.int32); sl = np.zeros(K + 1, np.int32)
    m = C.c_int32(0); tail = C.c_int32(0)
    f = lib().oracle_map_sequence
    f.restype = C.c_int32
    hits = f(C.c_void_p(cache._h), _p(vocab_map), C.c_int32(vocab_map.shape[0]), _p(d),
             C.c_int32(K), _p(q), _p(tgt), _p(qp), _p(ss), _p(sl), C.byref(m), C.byref(tail))
    mm = m.value
    return tgt[:mm].copy(), qp[:mm].copy(), ss[:mm + 1].copy(), sl[:mm].copy(), mm, tail.value, int(hits)


def softmax_row(row: np.ndarray, T: float) -> np.ndarray:
    """p(.) = softmax(row / T) in fp64; `row` float32, or uint16 bf16 bits."""
    row = np.ascontiguousarray(row)
    dt = DTYPE_F32 if row.dtype == np.float32 else DTYPE_BF16
    p = np.zeros(row.shape[0], dtype=np.float64)
    lib().oracle_softmax_row(_p(row), C.c_int32(dt), C.c_int64(row.shape[0]),
                             C.c_double(T), _p(p))
    return p


def full_mapping(q_row, vocab_map, v_p: int, first_draft_id: int, length: int,
                 ngram_token: int, ngram_prob: float) -> np.ndarray:
    """Eq. (2): q'(.) over the target vocabulary."""
    q_row = np.ascontiguousarray(q_row, dtype=np.float32)
    vocab_map = np.ascontiguousarray(vocab_map, dtype=np.int32)
    out = np.zeros(v_p, dtype=np.float64)
    lib().oracle_full_mapping(_p(q_row), C.c_int32(q_row.shape[0]), _p(vocab_map),
                              C.c_int64(v_p), C.c_int32(first_draft_id), C.c_int32(length),
                              C.c_int32(ngram_token), C.c_double(ngram_prob), _p(out))
    return out


def logits_to_numpy(t):
    """torch f32 / bf16 tensor (any device) -> (numpy array, oracle dtype code)."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float32:
        return t.numpy(), DTYPE_F32
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16), DTYPE_BF16
    raise TypeError(t.dtype)


def max_threads() -> int:
    return int(lib().oracle_openmp_threads())
