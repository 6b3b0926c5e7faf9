"""Pins for the oracle's Token Entropy (Section 3.2: e = -log P(x | context)).

The oracle is checked against closed forms, invariances of the softmax, and library
routines that compute the same quantity by another route (scipy's log_softmax, torch's
float64 cross-entropy).  A dropped max-shift, a wrong sign, Shannon entropy instead of
surprisal, log base 2, a wrong target index or a transposed stride each break one of them.
"""
import math

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2405_12528_b200 import workloads as wl


@pytest.mark.parametrize("V", [2, 7, 32000, 128256])
def test_uniform_row_gives_log_v(V):
    for c in (0.0, -3.5, 11.0):
        row = torch.full((V,), c, dtype=torch.float32)
        assert oracle.token_entropy(row, V // 2) == pytest.approx(math.log(V), rel=0, abs=1e-12)


def test_dominant_logit_gives_zero():
    row = torch.zeros(1000, dtype=torch.float32)
    row[123] = 80.0
    e = oracle.token_entropy(row, 123)
    assert 0.0 <= e < 1e-30
    # and the other tokens of that row are 80 nats away
    assert oracle.token_entropy(row, 5) == pytest.approx(80.0, abs=1e-12)


def test_two_token_row_separates_surprisal_from_shannon_entropy():
    # P = (1/4, 3/4): surprisals ln 4 and ln 4/3; the row's Shannon entropy is 0.5623...
    row = torch.tensor([0.0, math.log(3.0)], dtype=torch.float32)
    ln3_f32 = float(row[1])
    assert oracle.token_entropy(row, 0) == pytest.approx(math.log1p(math.exp(ln3_f32)), abs=1e-14)
    assert oracle.token_entropy(row, 0) == pytest.approx(math.log(4.0), abs=1e-7)
    assert oracle.token_entropy(row, 1) == pytest.approx(math.log(4.0 / 3.0), abs=1e-7)
    assert abs(oracle.token_entropy(row, 0) - 0.5623351446) > 0.5


def test_natural_log_not_base_two():
    row = torch.zeros(8, dtype=torch.float32)
    assert oracle.token_entropy(row, 0) == pytest.approx(3 * math.log(2.0), abs=1e-14)
    assert abs(oracle.token_entropy(row, 0) - 3.0) > 0.5


def test_shift_invariance_and_large_magnitudes():
    g = torch.Generator().manual_seed(1)
    row = torch.randn(513, generator=g, dtype=torch.float32) * 3
    base = oracle.token_entropy(row, 17)
    for c in (64.0, -128.0, 1024.0):     # exactly representable shifts keep the differences exact
        shifted = (row.double() + c).float()
        if torch.equal(shifted.double() - c, row.double()):
            assert oracle.token_entropy(shifted, 17) == pytest.approx(base, abs=1e-12)
    # no overflow for logits far outside exp's range
    big = torch.tensor([1000.0, 999.0, -1000.0])
    assert oracle.token_entropy(big, 0) == pytest.approx(math.log1p(math.exp(-1.0)), abs=1e-12)
    assert oracle.token_entropy(big, 2) == pytest.approx(2000.0 + math.log1p(math.exp(-1.0)), abs=1e-9)


def test_permuting_other_columns_changes_nothing_but_rounding():
    g = torch.Generator().manual_seed(2)
    row = torch.randn(4097, generator=g, dtype=torch.float32) * 2
    base = oracle.token_entropy(row, 0)
    perm = torch.cat([torch.zeros(1, dtype=torch.long), 1 + torch.randperm(4096, generator=g)])
    assert oracle.token_entropy(row[perm], 0) == pytest.approx(base, abs=1e-12)


def test_probabilities_of_a_row_sum_to_one():
    g = torch.Generator().manual_seed(3)
    row = torch.randn(50, generator=g, dtype=torch.float32) * 4
    total = math.fsum(math.exp(-oracle.token_entropy(row, v)) for v in range(50))
    assert total == pytest.approx(1.0, abs=1e-13)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_against_library_log_softmax(dtype):
    g = torch.Generator().manual_seed(4)
    logits = (torch.randn(37, 1531, generator=g) * 2.5).to(dtype)
    ids = torch.randint(0, 1531, (37,), generator=g, dtype=torch.int32)
    got = oracle.score(logits, ids)
    z = logits.double().numpy()
    lib1 = -scipy.special.log_softmax(z, axis=1)[np.arange(37), ids.numpy()]
    lib2 = torch.nn.functional.cross_entropy(logits.double(), ids.long(), reduction="none").numpy()
    ld = z.astype(np.longdouble)
    lib3 = (np.log(np.exp(ld - ld.max(1, keepdims=True)).sum(1)) + ld.max(1)
            - ld[np.arange(37), ids.numpy()]).astype(np.float64)
    for ref in (lib1, lib2, lib3):
        np.testing.assert_allclose(got.double().numpy(), ref, rtol=0, atol=2e-6)   # fp32 rounding of e
        np.testing.assert_array_equal(got.numpy(), ref.astype(np.float32))


def test_bf16_rows_are_read_by_their_bit_patterns():
    g = torch.Generator().manual_seed(5)
    logits = (torch.randn(5, 300, generator=g) * 2).to(torch.bfloat16)
    ids = torch.tensor([0, 299, 7, 150, 42], dtype=torch.int32)
    assert torch.equal(oracle.score(logits, ids), oracle.score(logits.float(), ids))


def test_row_stride_and_ignored_or_bad_ids():
    g = torch.Generator().manual_seed(6)
    wide = torch.randn(6, 140, generator=g)
    view = wide[:, :100]                         # row stride 140, V = 100
    ids = torch.tensor([3, -1, 99, 100, -7, 0], dtype=torch.int32)
    got = oracle.score(view, ids)
    ref = oracle.score(view.contiguous(), ids)
    assert torch.equal(got, ref)
    assert got[1] == 0.0 and got[3] == 0.0 and got[4] == 0.0
    scratch = torch.empty(6)
    n_bad = oracle.lib().oracle_score(view.data_ptr(), oracle.F32, 6, 100, 140,
                                      ids.data_ptr(), scratch.data_ptr())
    assert n_bad == 2                              # 100 and -7; -1 is the "no prediction" mark


def test_scores_of_the_synthetic_workload_have_two_populations():
    # the input recipe: boosted-column tokens are predictable, free draws are surprising
    w = wl.WORKLOADS["tiny"].scaled(new_tokens=64)
    logits = wl.make_logits(w, 0, 0, 0)
    ids_pred = wl.make_token_ids(w, 0, 0, 0, rho=1.0)
    ids_free = wl.make_token_ids(w, 0, 0, 0, rho=0.0)
    e_pred, e_free = oracle.score(logits, ids_pred), oracle.score(logits, ids_free)
    assert (e_pred >= 0).all() and (e_free >= 0).all()
    assert e_pred.median() + 3 < e_free.median()
