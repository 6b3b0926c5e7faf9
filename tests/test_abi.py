"""The C-ABI library: it loads, exports every declared symbol, and rejects bad arguments on
the host before touching a device (so these run without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2405_12528_b200 import binding as B
from paper_2405_12528_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    builder.build()
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
