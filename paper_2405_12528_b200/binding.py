"""ctypes binding of ``libsirllm.so``: same names as the C ABI, argument marshalling only.

Every function takes CUDA torch tensors (device memory owned by the caller), checks
dtypes and contiguity, passes raw pointers and the current CUDA stream to the library
and raises :class:`SirllmError` on a negative return code.  There is no CPU fallback:
if the library is missing or a tensor is not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsirllm.so")

F32, BF16, F16 = 0, 1, 2
OK, ERR_NULL, ERR_BAD_CONFIG, ERR_ALIGN, ERR_CUDA, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5
STATUS_TOKEN_RANGE, STATUS_OVERFLOW, STATUS_TIMEOUT, STATUS_BAD_KEEP = 1, 2, 4, 8
MAX_CAPACITY = 49152
POLICY_STREAM, POLICY_RANDOM, POLICY_INTERVAL = 1, 2, 3
ROPE_HALF, ROPE_INTERLEAVED = 0, 1

EXPORTS = ["sirllm_workspace_bytes", "sirllm_workspace_init", "sirllm_score", "sirllm_score_static",
           "sirllm_score_partial",
           "sirllm_score_pairs", "sirllm_step_pairs", "sirllm_decay_select", "sirllm_keep_policy", "sirllm_rerotate_keys",
           "sirllm_compact_kv", "sirllm_step", "sirllm_step_phases", "sirllm_step_host",
           "sirllm_selftest_bounded_wait", "sirllm_status", "sirllm_strerror",
           "sirllm_last_cuda_error"]

_DTYPE_CODE = {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}
_KV = (torch.bfloat16, torch.float16)


class SirllmError(RuntimeError):
    def __init__(self, code: int, detail: str = ""):
        self.code = code
        super().__init__(f"sirllm error {code}: {detail}")


class Config(ctypes.Structure):
    """Mirror of ``sirllm_config``."""
    _fields_ = [("n_streams", ctypes.c_int32), ("n_layers", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("capacity", ctypes.c_int32), ("budget", ctypes.c_int32),
                ("n_sink", ctypes.c_int32), ("n_recent", ctypes.c_int32),
                ("threshold", ctypes.c_int32), ("max_new", ctypes.c_int32),
                ("kv_dtype", ctypes.c_int32), ("logits_dtype", ctypes.c_int32),
                ("vocab", ctypes.c_int64), ("logits_row_stride", ctypes.c_int64)]

    @property
    def planes_per_stream(self) -> int:
        return self.n_layers * self.n_kv_heads


def make_config(n_streams, n_layers, n_kv_heads, head_dim, capacity, budget, n_sink, n_recent,
                max_new, vocab, logits_dtype, kv_dtype, threshold=None, logits_row_stride=None) -> Config:
    code = lambda d: _DTYPE_CODE[d] if isinstance(d, torch.dtype) else {"f32": F32, "bf16": BF16, "f16": F16}[d]
    return Config(n_streams, n_layers, n_kv_heads, head_dim, capacity, budget, n_sink, n_recent,
                  budget if threshold is None else threshold, max_new, code(kv_dtype),
                  code(logits_dtype), vocab, vocab if logits_row_stride is None else logits_row_stride)


def config_from_workload(w, **overrides) -> Config:
    """Config for a :class:`workloads.Workload`."""
    kw = dict(n_streams=w.n_streams, n_layers=w.n_layers, n_kv_heads=w.n_kv_heads,
              head_dim=w.head_dim, capacity=w.capacity, budget=w.budget, n_sink=w.n_sink,
              n_recent=w.n_recent, max_new=w.new_tokens, vocab=w.vocab,
              logits_dtype=w.logits_dtype, kv_dtype=w.kv_dtype, threshold=w.threshold)
    kw.update(overrides)
    return make_config(**kw)


_lib = None


def lib():
    """The loaded library; raises if it was not built (``python -m paper_2405_12528_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            # a source checkout: compile once with nvcc; without a compiler this fails loudly
            try:
                from . import build as _build
                _build.build()
            except Exception as exc:
                raise SirllmError(ERR_CUDA, f"{_LIB_PATH} is not built and could not be compiled "
                                            f"({exc}); run paper_2405_12528_b200/build.py") from exc
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, cfgp = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(Config)
        L.sirllm_workspace_bytes.restype = ctypes.c_size_t
        L.sirllm_workspace_bytes.argtypes = [cfgp]
        L.sirllm_workspace_init.restype = ctypes.c_int
        L.sirllm_workspace_init.argtypes = [cfgp, vp, vp]
        L.sirllm_score.restype = ctypes.c_int
        L.sirllm_score.argtypes = [cfgp, vp, vp, vp, vp, vp, vp]
        L.sirllm_score_static.restype = ctypes.c_int
        L.sirllm_score_static.argtypes = [cfgp, vp, vp, vp, vp, vp, vp]
        L.sirllm_score_partial.restype = ctypes.c_int
        L.sirllm_score_partial.argtypes = [cfgp, vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, vp, vp,
                                           vp, ctypes.c_int64, vp, vp, vp]
        L.sirllm_score_pairs.restype = ctypes.c_int
        L.sirllm_score_pairs.argtypes = [cfgp, vp, i32, ctypes.c_int64, vp, vp, vp, vp, vp, vp]
        L.sirllm_step_pairs.restype = ctypes.c_int
        L.sirllm_step_pairs.argtypes = [cfgp, vp, i32, ctypes.c_int64] + [vp] * 14
        L.sirllm_decay_select.restype = ctypes.c_int
        L.sirllm_decay_select.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, i32, vp, vp]
        L.sirllm_keep_policy.restype = ctypes.c_int
        L.sirllm_keep_policy.argtypes = [cfgp, i32, vp, ctypes.c_uint64, i32, i32, vp, vp, vp, vp]
        L.sirllm_rerotate_keys.restype = ctypes.c_int
        L.sirllm_rerotate_keys.argtypes = [cfgp, vp, vp, vp, ctypes.c_double, i32, vp]
        L.sirllm_compact_kv.restype = ctypes.c_int
        L.sirllm_compact_kv.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.sirllm_step.restype = ctypes.c_int
        L.sirllm_step.argtypes = [cfgp] + [vp] * 14
        L.sirllm_step_phases.restype = ctypes.c_int
        L.sirllm_step_phases.argtypes = [cfgp] + [vp] * 14 + [ctypes.POINTER(vp)]
        L.sirllm_step_host.restype = ctypes.c_int
        L.sirllm_step_host.argtypes = [cfgp] + [vp] * 23
        L.sirllm_selftest_bounded_wait.restype = ctypes.c_int
        L.sirllm_selftest_bounded_wait.argtypes = [cfgp, vp, ctypes.c_uint32, vp]
        L.sirllm_status.restype = ctypes.c_int
        L.sirllm_status.argtypes = [vp, vp, ctypes.POINTER(i32), i32]
        L.sirllm_strerror.restype = ctypes.c_char_p
        L.sirllm_strerror.argtypes = [ctypes.c_int]
        L.sirllm_last_cuda_error.restype = ctypes.c_char_p
        L.sirllm_last_cuda_error.argtypes = []
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != OK:
        L = lib()
        detail = L.sirllm_strerror(rc).decode()
        if rc == ERR_CUDA:
            detail += ": " + L.sirllm_last_cuda_error().decode()
        raise SirllmError(rc, detail)


class _Arg:
    """One tensor argument and what the configuration demands of it.  The C side sees plain
    pointers and no sizes, so every call checks ALL its arguments here first - dtype and
    element count, then residence (right kind of memory, contiguous, on the current device) -
    and only then hands out pointers."""

    def __init__(self, t, dtype, name, numel=0, host=False):
        self.t, self.dtype, self.name, self.numel, self.host = t, dtype, name, numel, host

    def check_shape(self):
        t = self.t
        if t is None:
            return
        if self.dtype is not None and t.dtype not in (self.dtype if isinstance(self.dtype, tuple) else (self.dtype,)):
            raise SirllmError(ERR_BAD_CONFIG, f"{self.name} has dtype {t.dtype}")
        if t.numel() < self.numel:
            raise SirllmError(ERR_BAD_CONFIG, f"{self.name} holds {t.numel()} elements, the "
                                              f"configuration needs {self.numel}")

    def check_residence(self):
        t = self.t
        if t is None:
            return
        if self.host:
            if t.is_cuda or not t.is_contiguous():
                raise SirllmError(ERR_ALIGN, f"{self.name} must be a contiguous host tensor")
            return
        if not t.is_cuda:
            raise SirllmError(ERR_NULL, f"{self.name} must be a CUDA tensor (there is no CPU path)")
        if not t.is_contiguous() and self.dtype is not None:
            raise SirllmError(ERR_ALIGN, f"{self.name} must be contiguous")
        if t.device.index != torch.cuda.current_device():
            raise SirllmError(ERR_BAD_CONFIG, f"{self.name} lives on {t.device}, the current device "
                                              f"is cuda:{torch.cuda.current_device()}")

    def ptr(self):
        return None if self.t is None else self.t.data_ptr()


def _dev(t, dtype=None, name="tensor", numel: int = 0) -> _Arg:
    return _Arg(t, dtype, name, numel)


class Prepared:
    """A call whose arguments were checked and marshalled once (see :func:`prepared`): calling
    it again costs one ctypes call.  It keeps its tensors alive and reads the current CUDA
    stream at every call; it must be called with the device it was prepared on current."""

    def __init__(self, fn, cfg, args):
        self._fn, self._cfg = fn, Config.from_buffer_copy(cfg)
        self._keep = [a.t for a in args if isinstance(a, _Arg)]
        self._raw = [a.ptr() if isinstance(a, _Arg) else a for a in args]
        self._stream_at = [i for i, a in enumerate(args) if isinstance(a, _CurrentStream)]
        self._cfg_ref = ctypes.byref(self._cfg)

    def __call__(self) -> None:
        raw = self._raw
        for i in self._stream_at:
            raw[i] = torch.cuda.current_stream().cuda_stream
        rc = self._fn(self._cfg_ref, *raw)
        if rc != OK:
            _check(rc)


_preparing = threading.local()


def prepared(func, *args, **kwargs) -> Prepared:
    """``prepared(sirllm_step, cfg, logits, ...)`` checks and marshals the arguments of one of
    this module's calls once and returns a :class:`Prepared` that issues exactly that call
    (same tensors, whatever they hold by then) each time it is invoked - for loops that repeat
    a call thousands of times a second, where the per-argument checks would dominate."""
    _preparing.out = None
    _preparing.on = True
    try:
        func(*args, **kwargs)
    finally:
        _preparing.on = False
    if _preparing.out is None:
        raise SirllmError(ERR_BAD_CONFIG, f"{getattr(func, '__name__', func)} cannot be prepared")
    return _preparing.out


def _call(fn, cfg, *args) -> None:
    """Checks every tensor argument (shapes of all first, then residence), then calls ``fn``
    (or, under :func:`prepared`, hands back the marshalled call instead of making it)."""
    for a in args:
        if isinstance(a, _Arg):
            a.check_shape()
    for a in args:
        if isinstance(a, _Arg):
            a.check_residence()
    if getattr(_preparing, "on", False):
        _preparing.out = Prepared(fn, cfg, args)
        return
    raw = [a.ptr() if isinstance(a, _Arg) else _stream_handle() if isinstance(a, _CurrentStream) else a
           for a in args]
    _check(fn(ctypes.byref(cfg), *raw))


class _CurrentStream:
    """Placeholder for the current CUDA stream's handle, looked up after the argument checks."""


def _stream() -> _CurrentStream:
    return _CurrentStream()


def _stream_handle() -> int:
    return torch.cuda.current_stream().cuda_stream


def _rows(cfg: Config) -> int:
    return cfg.n_streams * cfg.max_new


def _kv_numel(cfg: Config) -> int:
    return cfg.n_streams * cfg.n_layers * cfg.n_kv_heads * cfg.capacity * cfg.head_dim


class _KvArg(_Arg):
    def __init__(self, cfg, t, name):
        super().__init__(t, _KV, name, _kv_numel(cfg))
        self.code = cfg.kv_dtype

    def check_shape(self):
        super().check_shape()
        if self.t is not None and _DTYPE_CODE.get(self.t.dtype) != self.code:
            raise SirllmError(ERR_BAD_CONFIG, f"{self.name} dtype {self.t.dtype} does not match the config")


def _kv(cfg: Config, t, name) -> _Arg:
    return _KvArg(cfg, t, name)


def _ws(cfg: Config, ws) -> _Arg:
    return _dev(ws, torch.uint8, "ws", sirllm_workspace_bytes(cfg))


class _LogitsArg(_Arg):
    """A logits matrix [>= rows, vocab] whose rows are logits_row_stride elements apart
    (a column slice of a wider buffer is fine: only the last dimension must be dense)."""

    def __init__(self, cfg, t, name="logits", host=False):
        super().__init__(t, None, name, 0, host)
        self.cfg = cfg

    def check_shape(self):
        cfg, t = self.cfg, self.t
        if t is None:
            return
        if _DTYPE_CODE.get(t.dtype) != cfg.logits_dtype:
            raise SirllmError(ERR_BAD_CONFIG, f"{self.name} dtype {t.dtype} does not match the config")
        rows = _rows(cfg)
        if t.dim() != 2 or t.shape[1] != cfg.vocab or t.shape[0] < rows:
            raise SirllmError(ERR_BAD_CONFIG, f"{self.name} has shape {tuple(t.shape)}, the "
                                              f"configuration needs [>= {rows}, {cfg.vocab}]")
        if t.stride(1) != 1 or (t.shape[0] > 1 and t.stride(0) != cfg.logits_row_stride):
            raise SirllmError(ERR_ALIGN, f"{self.name} rows must be logits_row_stride elements apart")

    def check_residence(self):
        if self.host and self.t is not None:
            if self.t.is_cuda:
                raise SirllmError(ERR_ALIGN, f"{self.name} must be a host tensor")
            return
        super().check_residence()


def _logits(cfg: Config, logits) -> _Arg:
    return _LogitsArg(cfg, logits)


class _PairsArg(_Arg):
    """Per-tile (max, sum exp) pairs [>= rows, n_tiles, 2], fp32, pairs contiguous."""

    def __init__(self, cfg, t):
        super().__init__(t, None, "pairs")
        self.cfg = cfg

    def check_shape(self):
        t = self.t
        if t is None:
            raise SirllmError(ERR_NULL, "pairs is required")
        if t.dtype != torch.float32:
            raise SirllmError(ERR_BAD_CONFIG, "pairs must be float32")
        if t.dim() != 3 or t.shape[2] != 2 or t.stride(2) != 1 or t.stride(1) != 2:
            raise SirllmError(ERR_ALIGN, "pairs must be [rows, n_tiles, 2] with contiguous pairs")
        if t.shape[0] < _rows(self.cfg):
            raise SirllmError(ERR_BAD_CONFIG, f"pairs hold {t.shape[0]} rows, the configuration "
                                              f"needs {_rows(self.cfg)}")

    @property
    def n_tiles(self) -> int:
        return int(self.t.shape[1])

    @property
    def row_stride(self) -> int:
        return int(self.t.stride(0) // 2 if self.t.shape[0] > 1 else self.t.shape[1])


def sirllm_workspace_bytes(cfg: Config) -> int:
    return lib().sirllm_workspace_bytes(ctypes.byref(cfg))


def new_workspace(cfg: Config, device="cuda") -> torch.Tensor:
    """Allocates (with torch) and initialises a workspace for ``cfg``."""
    n = sirllm_workspace_bytes(cfg)
    if n == 0:
        raise SirllmError(ERR_BAD_CONFIG, "invalid configuration")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    sirllm_workspace_init(cfg, ws)
    return ws


def sirllm_workspace_init(cfg: Config, ws: torch.Tensor) -> None:
    _call(lib().sirllm_workspace_init, cfg, _ws(cfg, ws), _stream())


def _score_args(cfg: Config, token_ids, n_new, out_entropy):
    return (_dev(token_ids, torch.int32, "token_ids", _rows(cfg)),
            _dev(n_new, torch.int32, "n_new", cfg.n_streams),
            _dev(out_entropy, torch.float32, "out_entropy", _rows(cfg)))


def sirllm_score(cfg: Config, logits, token_ids, n_new, out_entropy, ws) -> None:
    _call(lib().sirllm_score, cfg, _logits(cfg, logits), *_score_args(cfg, token_ids, n_new, out_entropy),
          _ws(cfg, ws), _stream())


def sirllm_score_static(cfg: Config, logits, token_ids, n_new, out_entropy, status=None) -> None:
    """``sirllm_score`` without a workspace: for callers that cannot allocate device memory
    (the scratch is a fixed array inside the library; at most 16384 logits rows per call,
    and calls that overlap on the GPU race).  ``status``: optional int32 device word."""
    _call(lib().sirllm_score_static, cfg, _logits(cfg, logits),
          *_score_args(cfg, token_ids, n_new, out_entropy), _dev(status, torch.int32, "status", 1),
          _stream())


class _SliceArg(_Arg):
    """One rank's column range of the logits: [>= rows, n_cols], last dimension dense."""

    def __init__(self, cfg, t, col0):
        super().__init__(t, None, "logits_slice")
        self.cfg, self.col0 = cfg, int(col0)

    def check_shape(self):
        cfg, t = self.cfg, self.t
        if t is None:
            raise SirllmError(ERR_NULL, "logits_slice is required")
        if _DTYPE_CODE.get(t.dtype) != cfg.logits_dtype:
            raise SirllmError(ERR_BAD_CONFIG, f"logits_slice dtype {t.dtype} does not match the config")
        if t.dim() != 2 or t.shape[0] < _rows(cfg) or self.col0 < 0 or self.col0 + t.shape[1] > cfg.vocab:
            raise SirllmError(ERR_BAD_CONFIG, f"logits_slice has shape {tuple(t.shape)} at column "
                                              f"{self.col0}, the configuration needs [>= {_rows(cfg)}, "
                                              f"<= {cfg.vocab - self.col0}]")
        if t.shape[1] > 0 and t.stride(1) != 1:
            raise SirllmError(ERR_ALIGN, "logits_slice rows must be dense")

    @property
    def row_stride(self) -> int:
        t = self.t
        return int(t.stride(0)) if t.shape[0] > 1 and t.shape[1] > 0 else max(int(t.shape[1]), 1)


def sirllm_score_partial(cfg: Config, logits_slice, col0: int, token_ids, n_new, pairs_out, target_out,
                         ws, pair_column: int = 0) -> None:
    """One rank's share of vocabulary-parallel scoring: ``logits_slice`` holds columns
    ``[col0, col0 + n_cols)``; ``pairs_out`` is ``[rows, n_ranks, 2]`` fp32 and this call fills
    column ``pair_column`` of it; ``target_out`` is fp32 ``[rows]``."""
    sl = _SliceArg(cfg, logits_slice, col0)
    sl.check_shape()
    pa = _PairsArg(cfg, pairs_out)
    pa.check_shape()
    if not 0 <= pair_column < pa.n_tiles:
        raise SirllmError(ERR_BAD_CONFIG, f"pair_column {pair_column} outside [0, {pa.n_tiles})")
    ids, nn, tgt = _score_args(cfg, token_ids, n_new, target_out)
    tgt.name = "target_out"
    pa.check_residence()
    _call(lib().sirllm_score_partial, cfg, sl, int(col0), int(logits_slice.shape[1]), sl.row_stride,
          ids, nn, pairs_out.data_ptr() + 8 * int(pair_column), pa.row_stride, tgt, _ws(cfg, ws), _stream())


def sirllm_score_pairs(cfg: Config, pairs, target_logit, token_ids, n_new, out_entropy, ws) -> None:
    """Scores from per-tile ``(max, sum exp)`` pairs ``[rows, n_tiles, 2]`` and target logits."""
    pa = _PairsArg(cfg, pairs)
    pa.check_shape()
    _call(lib().sirllm_score_pairs, cfg, pa, pa.n_tiles, pa.row_stride,
          _dev(target_logit, torch.float32, "target_logit", _rows(cfg)),
          *_score_args(cfg, token_ids, n_new, out_entropy), _ws(cfg, ws), _stream())


def _state_args(cfg: Config, scores, serial, live_len, decay):
    per_slot = cfg.n_streams * cfg.capacity
    return (_dev(scores, torch.float32, "scores", per_slot),
            _dev(serial, torch.int64, "serial", per_slot),
            _dev(live_len, torch.int32, "live_len", cfg.n_streams),
            _dev(decay, torch.float32, "decay", cfg.n_streams))


def _keep_args(cfg: Config, keep_idx, n_keep):
    return (_dev(keep_idx, torch.int32, "keep_idx", cfg.n_streams * cfg.threshold),
            _dev(n_keep, torch.int32, "n_keep", cfg.n_streams))


def _round_args(cfg: Config, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx, n_keep,
                new_entropy, ws):
    """The arguments sirllm_step, _step_pairs, _step_phases and _step_host share, in ABI order."""
    ids, nn, ent = _score_args(cfg, token_ids, n_new, new_entropy)
    return (ids, nn) + _state_args(cfg, scores, serial, live_len, decay) + \
        (_kv(cfg, k, "k"), _kv(cfg, v, "v")) + _keep_args(cfg, keep_idx, n_keep) + (ent, _ws(cfg, ws))


def sirllm_step_pairs(cfg: Config, pairs, target_logit, token_ids, n_new, scores, serial, live_len,
                      decay, k, v, keep_idx, n_keep, new_entropy, ws) -> None:
    pa = _PairsArg(cfg, pairs)
    pa.check_shape()
    _call(lib().sirllm_step_pairs, cfg, pa, pa.n_tiles, pa.row_stride,
          _dev(target_logit, torch.float32, "target_logit", _rows(cfg)),
          *_round_args(cfg, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx, n_keep,
                       new_entropy, ws), _stream())


def sirllm_decay_select(cfg: Config, scores, serial, live_len, decay, keep_idx, n_keep,
                        compact_scores, ws) -> None:
    _call(lib().sirllm_decay_select, cfg, *_state_args(cfg, scores, serial, live_len, decay),
          *_keep_args(cfg, keep_idx, n_keep), int(bool(compact_scores)), _ws(cfg, ws), _stream())


def sirllm_keep_policy(cfg: Config, policy: int, live_len, seed: int, rnd: int, stream_base: int,
                       keep_idx, n_keep, ws) -> None:
    """Keep lists of StreamLLM / RandomLLM / IntervalLLM (``POLICY_*``) for ``sirllm_compact_kv``."""
    _call(lib().sirllm_keep_policy, cfg, int(policy), _dev(live_len, torch.int32, "live_len", cfg.n_streams),
          int(seed), int(rnd), int(stream_base), *_keep_args(cfg, keep_idx, n_keep), _ws(cfg, ws),
          _stream())


def sirllm_rerotate_keys(cfg: Config, k, keep_idx, n_keep, rope_base: float, layout: int) -> None:
    """Turns the moved rows of a compacted post-rotary K cache to their new positions."""
    _call(lib().sirllm_rerotate_keys, cfg, _kv(cfg, k, "k"), *_keep_args(cfg, keep_idx, n_keep),
          float(rope_base), int(layout), _stream())


def sirllm_compact_kv(cfg: Config, k_src, v_src, k_dst, v_dst, keep_idx, n_keep, ws) -> None:
    _call(lib().sirllm_compact_kv, cfg, _kv(cfg, k_src, "k_src"), _kv(cfg, v_src, "v_src"),
          _kv(cfg, k_dst, "k_dst"), _kv(cfg, v_dst, "v_dst"), *_keep_args(cfg, keep_idx, n_keep),
          _ws(cfg, ws), _stream())


def sirllm_step(cfg: Config, logits, token_ids, n_new, scores, serial, live_len, decay, k, v,
                keep_idx, n_keep, new_entropy, ws) -> None:
    _call(lib().sirllm_step, cfg, _logits(cfg, logits),
          *_round_args(cfg, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx, n_keep,
                       new_entropy, ws), _stream())


def sirllm_step_phases(cfg: Config, logits, token_ids, n_new, scores, serial, live_len, decay, k, v,
                       keep_idx, n_keep, new_entropy, ws, events) -> None:
    """``sirllm_step`` that records the four ``torch.cuda.Event`` objects in ``events``
    (created with ``enable_timing=True``) around its three phases."""
    handles = (ctypes.c_void_p * 4)()
    for i, ev in enumerate(events):
        if not ev.cuda_event:          # torch creates the handle lazily, on first record
            ev.record()
        handles[i] = ev.cuda_event
    _call(lib().sirllm_step_phases, cfg, _logits(cfg, logits),
          *_round_args(cfg, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx, n_keep,
                       new_entropy, ws), _stream(), handles)


def _host(t, dtype=None, name="tensor", numel: int = 0) -> _Arg:
    return _Arg(t, dtype, name, numel, host=True)


def sirllm_step_host(cfg: Config, h_logits, h_token_ids, h_n_new, h_new_k, h_new_v, h_live_len,
                     d_logits, d_token_ids, d_n_new, scores, serial, live_len, decay, k, v,
                     keep_idx, n_keep, new_entropy, h_keep_idx, h_n_keep, h_new_entropy, ws) -> None:
    """One round with HOST inputs and outputs (``h_*`` are CPU tensors, ideally pinned);
    the results are valid after ``torch.cuda.current_stream().synchronize()``."""
    rows, S = _rows(cfg), cfg.n_streams
    new_rows = S * cfg.n_layers * cfg.n_kv_heads * cfg.max_new * cfg.head_dim
    rest = _round_args(cfg, d_token_ids, d_n_new, scores, serial, live_len, decay, k, v, keep_idx,
                       n_keep, new_entropy, ws)
    _call(lib().sirllm_step_host, cfg, _LogitsArg(cfg, h_logits, "h_logits", host=True),
          _host(h_token_ids, torch.int32, "h_token_ids", rows), _host(h_n_new, torch.int32, "h_n_new", S),
          _host(h_new_k, _KV, "h_new_k", new_rows), _host(h_new_v, _KV, "h_new_v", new_rows),
          _host(h_live_len, torch.int32, "h_live_len", S), _LogitsArg(cfg, d_logits, "d_logits"),
          *rest[:-1], _host(h_keep_idx, torch.int32, "h_keep_idx", S * cfg.threshold),
          _host(h_n_keep, torch.int32, "h_n_keep", S),
          _host(h_new_entropy, torch.float32, "h_new_entropy", rows), rest[-1], _stream())


def sirllm_selftest_bounded_wait(cfg: Config, ws: torch.Tensor, polls: int = 2000) -> None:
    """Lets one device-side bounded wait run out on purpose (raises STATUS_TIMEOUT in ``ws``)."""
    _call(lib().sirllm_selftest_bounded_wait, cfg, _ws(cfg, ws), int(polls), _stream())


def sirllm_status(ws: torch.Tensor, clear: bool = False) -> int:
    """Synchronises the current stream and returns the device status word."""
    out = ctypes.c_int32(0)
    arg = _dev(ws, torch.uint8, "ws", 4)
    arg.check_shape()
    arg.check_residence()
    _check(lib().sirllm_status(arg.ptr(), _stream_handle(), ctypes.byref(out), int(clear)))
    return out.value


def sirllm_strerror(code: int) -> str:
    return lib().sirllm_strerror(code).decode()


def sirllm_last_cuda_error() -> str:
    return lib().sirllm_last_cuda_error().decode()
