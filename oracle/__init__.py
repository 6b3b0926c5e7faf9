"""ctypes front end of the CPU oracle (``sirllm_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Nothing on the product path may import this package: it is for the tests, the smoke
check and the benchmark's CPU-baseline leg.  Arguments are CPU torch tensors (or numpy
arrays); bf16 / fp16 tensors are passed by their 16-bit patterns.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
import subprocess

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sirllm_oracle.c")
_LIB = os.path.join(_HERE, "libsirllm_oracle.so")

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math",
                               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def _bind(path: str):
    """Load an oracle library and declare its C signatures."""
    if True:
        L = ctypes.CDLL(path)
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
        L.oracle_token_entropy.restype = ctypes.c_double
        L.oracle_token_entropy.argtypes = [vp, ctypes.c_int, i64, i32, vp]
        L.oracle_score.restype = ctypes.c_int
        L.oracle_score.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, vp]
        L.oracle_score_pairs.restype = ctypes.c_int
        L.oracle_score_pairs.argtypes = [vp, i64, i64, i64, vp, vp, i64, vp]
        L.oracle_range_pair.restype = None
        L.oracle_range_pair.argtypes = [vp, ctypes.c_int, i64, i64, i32, vp, vp]
        L.oracle_decay.restype = None
        L.oracle_decay.argtypes = [vp, i64, f32]
        L.oracle_order_key.restype = ctypes.c_uint32
        L.oracle_order_key.argtypes = [f32]
        L.oracle_select.restype = i32
        L.oracle_select.argtypes = [vp, i32, i32, i32, i32, i32, vp]
        L.oracle_gather_rows.restype = None
        L.oracle_gather_rows.argtypes = [vp, vp, i64, vp, i32]
        L.oracle_step.restype = i32
        L.oracle_step.argtypes = [vp, i32, vp, vp, vp, i32, f32, i32, i32, i32, i32, i32, vp, vp,
                                  i64, i64, vp]
        L.oracle_keep_stream.restype = i32
        L.oracle_keep_stream.argtypes = [i32, i32, i32, i32, vp]
        L.oracle_keep_interval.restype = i32
        L.oracle_keep_interval.argtypes = [i32, i32, i32, i32, i32, vp]
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_keep_random.restype = i32
        L.oracle_keep_random.argtypes = [i32, i32, i32, i32, i32, ctypes.c_uint64, i32, i32, vp]
        L.oracle_rope_rotate_f64.restype = None
        L.oracle_rope_rotate_f64.argtypes = [vp, i32, i32, ctypes.c_double, ctypes.c_int]
        L.oracle_round16.restype = ctypes.c_double
        L.oracle_round16.argtypes = [ctypes.c_double, ctypes.c_int]
        L.oracle_rerotate_plane.restype = None
        L.oracle_rerotate_plane.argtypes = [vp, ctypes.c_int, i32, vp, i32, ctypes.c_double, ctypes.c_int]
    return L


def lib():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


@contextlib.contextmanager
def use_library(path: str):
    """Temporarily route every call through another build of the oracle (the tests use this
    to check that their pins reject deliberately broken variants)."""
    global _lib
    saved = lib()
    _lib = _bind(path)
    try:
        yield
    finally:
        _lib = saved


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.device.type == "cpu" and x.is_contiguous()
    return x.data_ptr()


def _logits_dtype(logits: torch.Tensor) -> int:
    if logits.dtype == torch.float32:
        return F32
    if logits.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"logits dtype {logits.dtype} not supported")


def token_entropy(row: torch.Tensor, token_id: int) -> float:
    """Token Entropy of one token as a double (before rounding to fp32)."""
    row = row.contiguous()
    return lib().oracle_token_entropy(_ptr(row), _logits_dtype(row), row.numel(), int(token_id), None)


def score(logits: torch.Tensor, ids: torch.Tensor) -> torch.Tensor:
    """fp32 scores of the ``T`` rows of ``logits [T, V]`` (last dim contiguous)."""
    assert logits.dim() == 2 and logits.stride(1) == 1
    T, V = logits.shape
    ids = ids.to(torch.int32).contiguous()
    out = torch.empty(T, dtype=torch.float32)
    stride = logits.stride(0) if T > 1 else V
    lib().oracle_score(logits.data_ptr(), _logits_dtype(logits), T, V, stride, _ptr(ids), _ptr(out))
    return out


def score_pairs(pairs: torch.Tensor, target_logit: torch.Tensor, ids: torch.Tensor, vocab: int) -> torch.Tensor:
    """fp32 scores from per-tile (max, sum exp) pairs ``[T, n_tiles, 2]`` and the target logits."""
    assert pairs.dtype == torch.float32 and pairs.dim() == 3 and pairs.shape[2] == 2
    pairs = pairs.contiguous()
    T, n_tiles = pairs.shape[:2]
    target_logit = target_logit.to(torch.float32).contiguous()
    ids = ids.to(torch.int32).contiguous()
    out = torch.empty(T, dtype=torch.float32)
    lib().oracle_score_pairs(_ptr(pairs), T, n_tiles, n_tiles, _ptr(target_logit), _ptr(ids), vocab, _ptr(out))
    return out


def range_pairs(logits: torch.Tensor, ids: torch.Tensor, v0: int, v1: int):
    """What one rank of a vocabulary-parallel LM head contributes for its columns ``[v0, v1)``:
    fp32 pairs ``[T, 2]`` (max, sum exp) and the target logits ``[T]`` (0 where the token's
    column lies outside the range)."""
    assert logits.dim() == 2 and logits.stride(1) == 1
    T, V = logits.shape
    assert 0 <= v0 <= v1 <= V
    ids = ids.to(torch.int32).contiguous()
    pairs = torch.zeros(T, 2, dtype=torch.float32)
    target = torch.zeros(T, dtype=torch.float32)
    esz = logits.element_size()
    for t in range(T):
        lib().oracle_range_pair(logits.data_ptr() + t * logits.stride(0) * esz, _logits_dtype(logits),
                                v0, v1, int(ids[t]), pairs.data_ptr() + 8 * t, target.data_ptr() + 4 * t)
    return pairs, target


def decay(E: torch.Tensor, live_len: int, eta: float) -> None:
    """In place: ``E[:live_len] *= eta`` as single fp32 multiplies."""
    assert E.dtype == torch.float32
    lib().oracle_decay(_ptr(E), int(live_len), float(np.float32(eta)))


def order_key(x: float) -> int:
    return lib().oracle_order_key(float(np.float32(x)))


def select(E: torch.Tensor, live_len: int, n_sink: int, n_recent: int, budget: int,
           threshold: int | None = None) -> torch.Tensor:
    """Kept slots (ascending int32) for scores ``E[:live_len]``."""
    threshold = budget if threshold is None else threshold
    assert E.dtype == torch.float32
    keep = torch.empty(max(int(live_len), budget, 1), dtype=torch.int32)
    n = lib().oracle_select(_ptr(E), int(live_len), n_sink, n_recent, budget, threshold, _ptr(keep))
    if n < 0:
        raise ValueError("inconsistent selection parameters")
    return keep[:n].clone()


def gather_rows(src: torch.Tensor, keep: torch.Tensor) -> torch.Tensor:
    """``src[keep]`` for a ``[slots, ...]`` tensor, by memcpy of whole rows."""
    src = src.contiguous()
    keep = keep.to(torch.int32).contiguous()
    out = torch.empty((keep.numel(),) + tuple(src.shape[1:]), dtype=src.dtype)
    row_bytes = src[0].numel() * src.element_size() if src.shape[0] else 0
    lib().oracle_gather_rows(_ptr(src), _ptr(out), row_bytes, _ptr(keep), keep.numel())
    return out


STREAM, RANDOM, INTERVAL = 1, 2, 3


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*ctr)
    k = (ctypes.c_uint32 * 2)(*key)
    out = (ctypes.c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, out)
    return list(out)


def keep_policy(policy: int, live_len: int, n_sink: int, n_recent: int, budget: int,
                threshold: int | None = None, seed: int = 0, stream: int = 0, rnd: int = 0) -> torch.Tensor:
    """Keep list (ascending int32) of one of the paper's comparison policies (Section 4.1.1)."""
    threshold = budget if threshold is None else threshold
    keep = torch.empty(max(int(live_len), budget, 1), dtype=torch.int32)
    if policy == STREAM:
        n = lib().oracle_keep_stream(live_len, n_sink, budget, threshold, _ptr(keep))
    elif policy == INTERVAL:
        n = lib().oracle_keep_interval(live_len, n_sink, n_recent, budget, threshold, _ptr(keep))
    elif policy == RANDOM:
        n = lib().oracle_keep_random(live_len, n_sink, n_recent, budget, threshold, seed, stream, rnd,
                                     _ptr(keep))
    else:
        raise ValueError("unknown policy")
    return keep[:n].clone()


ROPE_HALF, ROPE_INTERLEAVED = 0, 1


def rope_rotate(row: torch.Tensor, delta: int, base: float, layout: int) -> torch.Tensor:
    """A float64 row turned by ``delta`` positions of rotary embedding (new tensor)."""
    out = row.to(torch.float64).contiguous().clone()
    lib().oracle_rope_rotate_f64(_ptr(out), out.numel(), int(delta), float(base), int(layout))
    return out


def round16(v: float, bf16: bool) -> float:
    return lib().oracle_round16(float(v), int(bf16))


def rerotate_plane(plane: torch.Tensor, keep: torch.Tensor, base: float, layout: int) -> torch.Tensor:
    """Copy of a K plane ``[slots, d]`` (bf16/fp16) whose rows j < len(keep) are turned by
    ``j - keep[j]`` positions."""
    assert plane.dtype in (torch.bfloat16, torch.float16) and plane.dim() == 2
    out = plane.contiguous().clone()
    keep = keep.to(torch.int32).contiguous()
    lib().oracle_rerotate_plane(_ptr(out), int(plane.dtype == torch.bfloat16), out.shape[1], _ptr(keep),
                                keep.numel(), float(base), int(layout))
    return out


class Stream:
    """State of one dialogue stream as the oracle keeps it (Algorithm 1's variables)."""

    def __init__(self, capacity: int, n_sink: int, n_recent: int, budget: int, threshold: int,
                 eta: float, k: torch.Tensor | None = None, v: torch.Tensor | None = None):
        self.capacity, self.n_sink, self.n_recent = capacity, n_sink, n_recent
        self.budget, self.threshold, self.eta = budget, threshold, float(np.float32(eta))
        self.E = torch.zeros(capacity, dtype=torch.float32)
        self.serial = torch.full((capacity,), -1, dtype=torch.int64)
        self.next_serial = ctypes.c_int64(0)
        self.live_len = 0
        self.k, self.v = k, v          # [planes, capacity, head_dim] or None
        self.keep = torch.empty(0, dtype=torch.int32)

    def step(self, new_e: torch.Tensor) -> torch.Tensor:
        """Append the round's scores (its K/V rows must already sit in the caches), decay,
        and evict if over the threshold.  Returns the kept-slot list of the round."""
        new_e = new_e.to(torch.float32).contiguous()
        T = new_e.numel()
        keep = torch.empty(max(self.capacity, 1), dtype=torch.int32)
        n_planes, row_bytes = 0, 0
        if self.k is not None:
            assert self.k.is_contiguous() and self.k.shape[1] == self.capacity
            n_planes = self.k.shape[0]
            row_bytes = self.k.shape[2] * self.k.element_size()
        n = lib().oracle_step(_ptr(new_e), T, _ptr(self.E), _ptr(self.serial),
                              ctypes.addressof(self.next_serial), self.live_len, self.eta,
                              self.capacity, self.n_sink, self.n_recent, self.budget,
                              self.threshold, _ptr(self.k), _ptr(self.v), n_planes, row_bytes,
                              _ptr(keep))
        if n < 0:
            raise ValueError("round does not fit the cache or parameters are inconsistent")
        self.live_len = n
        self.keep = keep[:n].clone()
        return self.keep
