"""The C-ABI library: it loads, exports every declared symbol, and rejects bad arguments on
the host before touching a device (so these run without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2405_12528_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib(cuda_library):
    return B.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "sirllm.h")).read()
    declared = set(re.findall(r"\b(sirllm_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_config_struct_layout_matches_the_header():
    assert ctypes.sizeof(B.Config) == 12 * 4 + 2 * 8
    assert B.Config.vocab.offset == 48 and B.Config.logits_row_stride.offset == 56


def _cfg(**kw):
    base = dict(n_streams=1, n_layers=2, n_kv_heads=2, head_dim=64, capacity=1024, budget=256,
                n_sink=4, n_recent=64, max_new=512, vocab=32000, logits_dtype="f32", kv_dtype="f16")
    base.update(kw)
    return B.make_config(**base)


def test_workspace_size_is_pure_and_zero_for_bad_configs(lib):
    n = B.sirllm_workspace_bytes(_cfg())
    assert n > 0 and n % 256 == 0 and n == B.sirllm_workspace_bytes(_cfg())
    assert B.sirllm_workspace_bytes(_cfg(max_new=1024)) > n
    for bad in (dict(budget=60), dict(threshold=100), dict(capacity=200), dict(head_dim=12), dict(head_dim=520),
                dict(capacity=B.MAX_CAPACITY + 1), dict(n_streams=0), dict(vocab=0),
                dict(logits_row_stride=31999), dict(logits_dtype="f16"), dict(kv_dtype="f32"),
                dict(n_sink=-1)):
        assert B.sirllm_workspace_bytes(_cfg(**bad)) == 0, bad


def test_host_side_argument_checks_return_codes(lib):
    cfg = _cfg()
    c = ctypes.byref(cfg)
    ws, p = 0x1000, 0x2000       # never dereferenced: the checks below fail first
    assert lib.sirllm_score(c, None, p, None, p, ws, None) == B.ERR_NULL
    assert lib.sirllm_score(c, p, p, None, p, None, None) == B.ERR_NULL
    assert lib.sirllm_score(c, p, p, None, p, ws + 8, None) == B.ERR_ALIGN
    assert lib.sirllm_score(c, p + 2, p, None, p, ws, None) == B.ERR_ALIGN
    assert lib.sirllm_score(None, p, p, None, p, ws, None) == B.ERR_NULL
    assert lib.sirllm_decay_select(c, p, None, p, p, None, p, 0, ws, None) == B.ERR_NULL
    assert lib.sirllm_compact_kv(c, p, None, None, None, p, p, ws, None) == B.ERR_NULL
    assert lib.sirllm_compact_kv(c, p + 4, None, p + 4, None, p, p, ws, None) == B.ERR_ALIGN
    assert lib.sirllm_compact_kv(c, p, p + 64, p, p + 128, p, p, ws, None) == B.ERR_BAD_CONFIG
    bad = _cfg(budget=10)
    assert lib.sirllm_step(ctypes.byref(bad), *([p] * 13), ws, None) == B.ERR_BAD_CONFIG
    assert lib.sirllm_status(None, None, None, 0) == B.ERR_NULL
    assert "NULL" in B.sirllm_strerror(B.ERR_NULL)
    assert B.sirllm_strerror(0) == "ok"


def test_binding_refuses_cpu_tensors(lib):
    import torch
    cfg = _cfg()
    with pytest.raises(B.SirllmError):
        B.sirllm_score(cfg, torch.zeros(512, 32000), torch.zeros(512, dtype=torch.int32), None,
                       torch.zeros(512), torch.zeros(1024, dtype=torch.uint8))


def test_binding_refuses_undersized_buffers_before_calling_the_library(lib):
    # the C side sees plain pointers: sizes are checked here, on the host, for every argument
    # (CPU tensors stand in: the size check comes before the residence check)
    import torch
    cfg = _cfg(n_streams=2, max_new=8, capacity=64, budget=16, n_sink=2, n_recent=2, vocab=100)
    rows, S, C = 16, 2, 64
    z = lambda n, dt=torch.float32: torch.zeros(n, dtype=dt)
    ws_ok = torch.zeros(B.sirllm_workspace_bytes(cfg), dtype=torch.uint8)
    logits = torch.zeros(rows, 100)
    ids, out = z(rows, torch.int32), z(rows)

    def refused(fn, *a, needle="needs"):
        with pytest.raises(B.SirllmError) as err:
            fn(*a)
        assert needle in str(err.value), str(err.value)

    refused(B.sirllm_score, cfg, logits, z(rows - 1, torch.int32), None, out, ws_ok)
    refused(B.sirllm_score, cfg, logits, ids, None, z(rows - 1), ws_ok)
    refused(B.sirllm_score, cfg, logits, ids, z(1, torch.int32), out, ws_ok)
    refused(B.sirllm_score, cfg, logits, ids, None, out, ws_ok[:-256])
    refused(B.sirllm_score, cfg, logits[:rows - 1], ids, None, out, ws_ok)          # too few rows
    refused(B.sirllm_score, cfg, torch.zeros(rows, 99), ids, None, out, ws_ok)      # wrong vocab
    refused(B.sirllm_score, cfg, logits.to(torch.bfloat16), ids, None, out, ws_ok, needle="dtype")
    refused(B.sirllm_decay_select, cfg, z(S * C - 1), None, z(S, torch.int32), z(S), z(S * 16, torch.int32),
            z(S, torch.int32), 1, ws_ok)
    refused(B.sirllm_decay_select, cfg, z(S * C), z(S * C - 1, torch.int64), z(S, torch.int32), z(S),
            z(S * 16, torch.int32), z(S, torch.int32), 1, ws_ok)
    refused(B.sirllm_decay_select, cfg, z(S * C), None, z(S, torch.int32), z(S), z(S * 16 - 1, torch.int32),
            z(S, torch.int32), 1, ws_ok)
    kv = torch.zeros(S, 4, C, 64, dtype=torch.float16)
    refused(B.sirllm_compact_kv, cfg, kv[:, :3], None, kv[:, :3], None, z(S * 16, torch.int32),
            z(S, torch.int32), ws_ok)
    refused(B.sirllm_compact_kv, cfg, kv.to(torch.bfloat16), None, kv.to(torch.bfloat16), None,
            z(S * 16, torch.int32), z(S, torch.int32), ws_ok, needle="dtype")
    # right sizes: the call gets as far as the residence check
    refused(B.sirllm_score, cfg, logits, ids, None, out, ws_ok, needle="CUDA tensor")


def test_step_host_checks_every_argument_before_its_first_copy(lib):
    # valid first stream, bad second stream: the call must be refused as a whole.  A refusal
    # that came after stream 0's copies had been enqueued would show up here as a CUDA error
    # (no device in this process), not as the argument error.
    cfg = _cfg(n_streams=2, max_new=8, capacity=64, budget=16, n_sink=2, n_recent=2, vocab=100)
    c = ctypes.byref(cfg)
    i32x2 = ctypes.c_int32 * 2
    host = (ctypes.c_char * (2 * 8 * 100 * 4))()
    ids = (ctypes.c_int32 * 16)()
    ws, p = 0x1000, 0x2000
    hp = ctypes.cast(host, ctypes.c_void_p)
    ip = ctypes.cast(ids, ctypes.c_void_p)

    def call(n_new, live, ws=ws, scores=p):
        a, b = i32x2(*n_new), i32x2(*live)
        return lib.sirllm_step_host(c, hp, ip, ctypes.cast(a, ctypes.c_void_p), None, None,
                                    ctypes.cast(b, ctypes.c_void_p), p, p, p, scores, None, p, p, p, p,
                                    p, p, p, hp, hp, hp, ws, None)

    assert call([4, 9], [0, 0]) == B.ERR_BAD_CONFIG          # n_new[1] > max_new
    assert call([4, -1], [0, 0]) == B.ERR_BAD_CONFIG
    assert call([4, 4], [0, -3]) == B.ERR_BAD_CONFIG         # negative length in stream 1
    assert call([4, 4], [0, 0], ws=ws + 8) == B.ERR_ALIGN    # the round's own checks come first too
    assert call([4, 4], [0, 0], scores=None) == B.ERR_NULL
