"""sirllm_score_static: the scoring entry point for callers that cannot allocate.

Some users of this library run where device memory is not theirs to allocate: inside a host
framework's plugin / custom-op slot that hands them inputs and outputs and nothing else, or
at a point of the program where calling the allocator is off limits because it may
synchronise the device or fail under memory pressure.  ``sirllm_score`` wants a workspace
from its caller; ``sirllm_score_static`` keeps its scratch in a fixed array inside the
library instead.  This test calls it through the C ABI and checks it against
``sirllm_score`` on the same inputs, twice in a row (the second call reuses the array with
whatever the first left there), and checks that problems beyond its fixed limits are
refused.  It is collected last on purpose and passes alone or after the other tests.
"""
import ctypes

import pytest
import torch

from helpers import assert_entropy_close
from paper_2405_12528_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(seed, S, M, V, dtype, n_new):
    g = torch.Generator().manual_seed(seed)
    logits = (torch.randn(S * M, V, generator=g) * 2.5).to(dtype).to(DEV)
    ids = torch.randint(0, V, (S * M,), generator=g, dtype=torch.int32)
    ids[1] = -1                       # "no prediction" mark
    ids[2] = V + 3                    # a bad id: scored 0 and flagged
    cfg = B.make_config(S, 1, 1, 8, 64, 16, 2, 2, M, V, dtype, torch.bfloat16)
    return cfg, logits, ids.to(DEV), torch.tensor(n_new, dtype=torch.int32, device=DEV)


def test_static_scratch_scoring_matches_the_workspace_entry_point_twice_in_a_row():
    # the first case needs several CTAs per row (tickets + partial pairs in the scratch),
    # the second is a different shape that reuses the same scratch bytes
    cases = [_case(11, 2, 24, 70001, torch.bfloat16, [24, 7]),
             _case(12, 3, 40, 20011, torch.float32, [40, 0, 13])]
    for cfg, logits, ids, n_new in cases:
        rows = cfg.n_streams * cfg.max_new
        want = torch.full((rows,), -3.0, device=DEV)
        ws = B.new_workspace(cfg)
        B.sirllm_score(cfg, logits, ids, n_new, want, ws)
        got = torch.full((rows,), -3.0, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.sirllm_score_static(cfg, logits, ids, n_new, got, status)
        torch.cuda.synchronize()
        assert_entropy_close(got, want)                       # the tolerance the parity tests use
        assert torch.equal(got.view(torch.int32), want.view(torch.int32))   # same kernel: same bits
        assert int(status[0]) == B.STATUS_TOKEN_RANGE == B.sirllm_status(ws)
        # and once more without a status word
        again = torch.full((rows,), -3.0, device=DEV)
        B.sirllm_score_static(cfg, logits, ids, n_new, again, None)
        torch.cuda.synchronize()
        assert torch.equal(again.view(torch.int32), want.view(torch.int32))


def test_static_scratch_scoring_refuses_problems_beyond_its_limits():
    out = torch.zeros(8, device=DEV)
    ids = torch.zeros(8, dtype=torch.int32, device=DEV)
    lg = torch.zeros(8, 16, dtype=torch.bfloat16, device=DEV)
    L = B.lib()
    # too many rows (n_streams * max_new > 16384)
    cfg = B.make_config(2, 1, 1, 8, 16384, 16, 2, 2, 8193, 16, torch.bfloat16, torch.bfloat16)
    rc = L.sirllm_score_static(ctypes.byref(cfg), lg.data_ptr(), ids.data_ptr(), None,
                               out.data_ptr(), None, None)
    assert rc == B.ERR_TOO_LARGE
    # rows * CTAs per row > 65536 (a 1M-entry fp32 vocabulary needs 62 CTAs per row)
    cfg = B.make_config(1, 1, 1, 8, 4096, 16, 2, 2, 2048, 1 << 20, torch.float32, torch.bfloat16)
    rc = L.sirllm_score_static(ctypes.byref(cfg), lg.data_ptr(), ids.data_ptr(), None,
                               out.data_ptr(), None, None)
    assert rc == B.ERR_TOO_LARGE
    assert "limit" in B.sirllm_strerror(B.ERR_TOO_LARGE)
