"""Seeded synthetic inputs for the retention pass: logits, token ids, K/V rows, decay ratios.

This module only *draws inputs*.  It contains none of the method's arithmetic (no
log-softmax, no decay, no selection, no gather) and is the one piece of code that
both the CUDA path's tests and the CPU oracle's tests may use.  Everything is a
pure function of integer keys, built from 32-bit integer hashing carried out with
torch integer ops, so the same call gives bit-identical tensors on ``cpu`` and on
``cuda`` (integer ops are exact; the few floating-point ops are single IEEE
multiplies/adds and round-to-nearest-even casts, which agree on both).

The inputs stand in for the dialogue streams and LM-head outputs of the paper's
experiments (Section 4: DailyDialog, Grocery Shopping, Rock-Paper-Scissors with
Vicuna / Yi models); neither the datasets nor the weights are used.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

_M32 = 0xFFFFFFFF
_GOLD = 0x9E3779B9

# tags that separate the random streams of the different inputs
TAG_LOGIT, TAG_BOOST, TAG_COIN, TAG_TOKEN, TAG_K, TAG_V, TAG_DECAY, TAG_LEN, TAG_PICK = range(1, 10)


def mix32(x: torch.Tensor) -> torch.Tensor:
    """Invertible 32-bit integer finaliser (two xor-shift-multiply rounds).

    ``x`` is an int64 tensor holding values in [0, 2**32); so is the result.
    """
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def fold(h: torch.Tensor, v) -> torch.Tensor:
    """Absorb the integer(s) ``v`` into the hash state ``h`` (broadcasting)."""
    if not torch.is_tensor(v):
        v = torch.tensor(int(v) & _M32, dtype=torch.int64, device=h.device)
    return mix32((h * 0x01000193 + (v & _M32) + _GOLD) & _M32)


def root_key(seed: int, tag: int, device) -> torch.Tensor:
    h = torch.tensor((int(seed) * 0x85EBCA6B + int(tag) * 0xC2B2AE35 + 1) & _M32,
                     dtype=torch.int64, device=device)
    return mix32(h)


def approx_normal(key: torch.Tensor, n_mix: int = 3) -> torch.Tensor:
    """Approximately standard-normal fp32 values, one per key.

    Sum of ``2 * n_mix`` independent 16-bit uniforms (Irwin-Hall), centred and
    scaled to unit variance; the tails stop at ``sqrt(6 * n_mix)`` sigma.  The
    integer sum is exact and the scaling is one fp32 multiply.
    """
    total = torch.zeros_like(key)
    for j in range(n_mix):
        u = mix32((key + (j + 1) * _GOLD) & _M32)
        total = total + (u & 0xFFFF) + (u >> 16)
    centred = (total - n_mix * 65535).to(torch.float32)
    var = 2 * n_mix * (65536.0 ** 2 - 1.0) / 12.0
    scale = torch.tensor(1.0 / math.sqrt(var), dtype=torch.float32, device=key.device)
    return centred * scale


def uniform_int(key: torch.Tensor, n: int) -> torch.Tensor:
    """Integers in [0, n) (int64) from 32-bit keys (modulo bias < n / 2**32)."""
    return mix32((key + _GOLD) & _M32) % int(n)


def uniform_unit(key: torch.Tensor) -> torch.Tensor:
    """fp32 uniforms in [0, 1): the top 24 bits of a hash, scaled by 2**-24."""
    return (mix32((key + _GOLD) & _M32) >> 8).to(torch.float32) * (1.0 / 16777216.0)


# --------------------------------------------------------------------------------------
# workload descriptions
# --------------------------------------------------------------------------------------

_DTYPES = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one synthetic streaming workload (all sizes per stream)."""

    name: str
    n_streams: int
    n_layers: int
    n_kv_heads: int
    head_dim: int
    capacity: int          # physical slots per plane
    budget: int            # retained cache size after an eviction
    n_sink: int
    n_recent: int
    new_tokens: int        # tokens appended per round
    vocab: int
    logits_dtype: str      # "f32" | "bf16"
    kv_dtype: str          # "f16" | "bf16"
    decay: float           # decay ratio; per-stream draw in [decay, decay_hi] if decay_hi set
    rounds: int
    decay_hi: Optional[float] = None
    zipf_bias: float = 0.0  # exponent s of the rank bias -s*ln(rank); 0 = none
    rho: float = 0.5        # share of rows whose realised token is the boosted column
    sigma: float = 2.0
    boost: float = 8.0

    @property
    def threshold(self) -> int:
        return self.budget

    @property
    def planes_per_stream(self) -> int:
        """(layer, kv-head) pairs of ONE of K or V for one stream."""
        return self.n_layers * self.n_kv_heads

    @property
    def row_bytes(self) -> int:
        return self.head_dim * 2

    @property
    def torch_logits_dtype(self):
        return _DTYPES[self.logits_dtype]

    @property
    def torch_kv_dtype(self):
        return _DTYPES[self.kv_dtype]

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five shapes the build is measured on.  "tiny" finishes on the CPU in seconds.
WORKLOADS = {
    "tiny": Workload("tiny", 1, 2, 8, 64, 1024, 256, 4, 64, 512, 32000, "f32", "f16", 0.9, 1),
    "llama2_7b": Workload("llama2_7b", 1, 32, 32, 128, 4096, 2048, 4, 256, 2048, 32000,
                          "bf16", "bf16", 0.9, 20),
    "mistral_7b_gqa": Workload("mistral_7b_gqa", 1, 32, 8, 128, 8192, 4096, 4, 512, 1024, 32000,
                               "bf16", "bf16", 0.8, 50),
    "llama3_8b": Workload("llama3_8b", 1, 32, 8, 128, 16384, 8192, 4, 1024, 4096, 128256,
                          "bf16", "bf16", 0.9, 20, zipf_bias=1.1),
    "batched64": Workload("batched64", 64, 32, 32, 128, 2048, 1024, 4, 256, 256, 32000,
                          "bf16", "bf16", 0.7, 100, decay_hi=1.0),
    # A quarter of llama3_8b in tokens and slots (same vocabulary, planes and row size): the
    # small case profiler captures run on.
    "llama3_8b_quarter": Workload("llama3_8b_quarter", 1, 32, 8, 128, 4096, 2048, 4, 256, 1024,
                                  128256, "bf16", "bf16", 0.9, 20, zipf_bias=1.1),
    # Shapes the paper's own runs had (Tables 1-3, 5-7): small rounds, no recent window.
    "rps_1024": Workload("rps_1024", 1, 32, 32, 128, 1152, 1024, 4, 0, 54, 32000,
                         "bf16", "bf16", 0.8, 2000),
    "dailydialog_512": Workload("dailydialog_512", 1, 32, 32, 128, 640, 512, 4, 0, 120, 32000,
                                "bf16", "bf16", 0.7, 4),
}


# --------------------------------------------------------------------------------------
# generators
# --------------------------------------------------------------------------------------

def zipf_bias_table(vocab: int, s: float, device="cpu") -> torch.Tensor:
    """fp32 table ``-s * ln(rank)``, rank = token id + 1, computed in double on the host."""
    rank = torch.arange(1, vocab + 1, dtype=torch.float64)
    return (-float(s) * torch.log(rank)).to(torch.float32).to(device)


def boosted_columns(w: Workload, seed: int, stream: int, rnd: int, n_rows: int, device) -> torch.Tensor:
    """The one column per logits row that receives the ``+boost`` bump (int64 [n_rows])."""
    h = fold(fold(root_key(seed, TAG_BOOST, device), stream), rnd)
    rows = torch.arange(n_rows, dtype=torch.int64, device=device)
    return uniform_int(fold(h, rows), w.vocab)


def make_logits(w: Workload, seed: int, stream: int, rnd: int, n_rows: Optional[int] = None,
                device="cpu", bias: Optional[torch.Tensor] = None,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Logits ``[n_rows, vocab]`` in the workload's dtype.

    ``z[t, v] = sigma * n(t, v) (+ bias[v])`` and one boosted column per row; rounded
    once (to nearest even) to the storage dtype.
    """
    n_rows = w.new_tokens if n_rows is None else n_rows
    dt = w.torch_logits_dtype
    if out is None:
        out = torch.empty((n_rows, w.vocab), dtype=dt, device=device)
    if n_rows == 0:
        return out
    if w.zipf_bias and bias is None:
        bias = zipf_bias_table(w.vocab, w.zipf_bias, device)
    h = fold(fold(root_key(seed, TAG_LOGIT, device), stream), rnd)
    cols = torch.arange(w.vocab, dtype=torch.int64, device=device)
    bcol = boosted_columns(w, seed, stream, rnd, n_rows, device)
    sigma = torch.tensor(w.sigma, dtype=torch.float32, device=device)
    step = max(1, (1 << 24) // w.vocab)
    for r0 in range(0, n_rows, step):
        r1 = min(n_rows, r0 + step)
        rows = torch.arange(r0, r1, dtype=torch.int64, device=device)
        hr = fold(h, rows)                                   # [r]
        key = fold(hr[:, None], cols[None, :])               # [r, V]
        z = approx_normal(key) * sigma
        if bias is not None:
            z = z + bias[None, :]
        z[torch.arange(r1 - r0, device=device), bcol[r0:r1]] += w.boost
        out[r0:r1] = z.to(dt)
    return out


def make_token_ids(w: Workload, seed: int, stream: int, rnd: int, n_rows: Optional[int] = None,
                   device="cpu", rho: Optional[float] = None) -> torch.Tensor:
    """Realised token ids (int32 [n_rows]).

    With probability ``rho`` the id is the row's boosted column (a predictable token),
    otherwise an independent uniform draw (a surprising token).
    """
    n_rows = w.new_tokens if n_rows is None else n_rows
    rho = w.rho if rho is None else rho
    rows = torch.arange(n_rows, dtype=torch.int64, device=device)
    bcol = boosted_columns(w, seed, stream, rnd, n_rows, device)
    hc = fold(fold(root_key(seed, TAG_COIN, device), stream), rnd)
    ht = fold(fold(root_key(seed, TAG_TOKEN, device), stream), rnd)
    coin = uniform_unit(fold(hc, rows))
    free = uniform_int(fold(ht, rows), w.vocab)
    ids = torch.where(coin < rho, bcol, free)
    return ids.to(torch.int32)


def make_kv_rows(w: Workload, seed: int, which: str, stream: int, serials: torch.Tensor,
                 planes: Optional[torch.Tensor] = None, device="cpu") -> torch.Tensor:
    """K or V rows ``[n_planes, n_serials, head_dim]`` in the workload's KV dtype.

    Element ``c`` of the row of token ``serial`` in plane ``p`` of stream ``s`` depends
    only on ``(which, s, p, serial, c)``, so a row can be recognised by its content
    wherever compaction moves it.
    """
    tag = TAG_K if which == "k" else TAG_V
    if planes is None:
        planes = torch.arange(w.planes_per_stream, dtype=torch.int64, device=device)
    planes = planes.to(device=device, dtype=torch.int64)
    serials = serials.to(device=device, dtype=torch.int64)
    dt = w.torch_kv_dtype
    out = torch.empty((planes.numel(), serials.numel(), w.head_dim), dtype=dt, device=device)
    if out.numel() == 0:
        return out
    h = fold(root_key(seed, tag, device), stream)
    cols = torch.arange(w.head_dim, dtype=torch.int64, device=device)
    hs = fold(h, serials)                                            # [S]
    step = max(1, (1 << 24) // max(1, serials.numel() * w.head_dim))
    for p0 in range(0, planes.numel(), step):
        p1 = min(planes.numel(), p0 + step)
        hp = fold(hs[None, :], planes[p0:p1, None])                  # [p, S]
        key = fold(hp[:, :, None], cols[None, None, :])              # [p, S, D]
        out[p0:p1] = approx_normal(key, n_mix=1).to(dt)
    return out


def stream_decay(w: Workload, seed: int, device="cpu") -> torch.Tensor:
    """Per-stream decay ratios (fp32 [n_streams])."""
    if w.decay_hi is None:
        return torch.full((w.n_streams,), w.decay, dtype=torch.float32, device=device)
    s = torch.arange(w.n_streams, dtype=torch.int64, device=device)
    u = uniform_unit(fold(root_key(seed, TAG_DECAY, device), s))
    lo = torch.tensor(w.decay, dtype=torch.float32, device=device)
    span = torch.tensor(w.decay_hi - w.decay, dtype=torch.float32, device=device)
    return lo + span * u


def ragged_lengths(seed: int, n_streams: int, rnd: int, max_new: int, device="cpu") -> torch.Tensor:
    """A ragged mix of per-stream round lengths in [0, max_new] (int32 [n_streams])."""
    s = torch.arange(n_streams, dtype=torch.int64, device=device)
    h = fold(fold(root_key(seed, TAG_LEN, device), rnd), s)
    return uniform_int(h, max_new + 1).to(torch.int32)


def random_scores(seed: int, n: int, device="cpu", quantise: int = 0) -> torch.Tensor:
    """Non-negative fp32 test scores; ``quantise`` > 0 forces many exact ties."""
    i = torch.arange(n, dtype=torch.int64, device=device)
    h = fold(root_key(seed, TAG_PICK, device), i)
    if quantise:
        return uniform_int(h, quantise).to(torch.float32) * 0.25
    return uniform_unit(h) * 12.0
