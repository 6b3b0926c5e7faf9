"""Pins for the oracle's rotary re-indexing of keys (Section 3.3, positions inside the cache)."""
import math

import numpy as np
import pytest
import torch

import oracle

LAYOUTS = [oracle.ROPE_HALF, oracle.ROPE_INTERLEAVED]


def _pairs(row, layout):
    d = row.numel()
    if layout == oracle.ROPE_HALF:
        return row[:d // 2].numpy() + 1j * row[d // 2:].numpy()
    return row[0::2].numpy() + 1j * row[1::2].numpy()


@pytest.mark.parametrize("layout", LAYOUTS)
def test_rotation_is_complex_multiplication_by_a_unit_phasor(layout):
    # library route: numpy complex arithmetic, theta_i = base^(-2i/d)
    g = torch.Generator().manual_seed(1)
    d, base = 64, 10000.0
    row = torch.randn(d, generator=g, dtype=torch.float64)
    for delta in (1, -3, 17, -4096, 12345):
        got = _pairs(oracle.rope_rotate(row, delta, base, layout), layout)
        theta = base ** (-2.0 * np.arange(d // 2) / d)
        want = _pairs(row, layout) * np.exp(1j * delta * theta)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)


def test_one_pair_one_radian():
    # d = 2: a single pair with theta_0 = 1
    out = oracle.rope_rotate(torch.tensor([1.0, 0.0]), 1, 500.0, oracle.ROPE_HALF)
    assert out.tolist() == pytest.approx([math.cos(1.0), math.sin(1.0)], abs=1e-15)
    out = oracle.rope_rotate(torch.tensor([0.0, 2.0]), -1, 500.0, oracle.ROPE_INTERLEAVED)
    assert out.tolist() == pytest.approx([2 * math.sin(1.0), 2 * math.cos(1.0)], abs=1e-15)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_group_properties_and_norms(layout):
    g = torch.Generator().manual_seed(2)
    row = torch.randn(128, generator=g, dtype=torch.float64)
    assert torch.equal(oracle.rope_rotate(row, 0, 10000.0, layout), row)
    a = oracle.rope_rotate(oracle.rope_rotate(row, 37, 10000.0, layout), -12, 10000.0, layout)
    assert torch.allclose(a, oracle.rope_rotate(row, 25, 10000.0, layout), atol=1e-12, rtol=0)
    back = oracle.rope_rotate(oracle.rope_rotate(row, 999, 10000.0, layout), -999, 10000.0, layout)
    assert torch.allclose(back, row, atol=1e-12, rtol=0)
    np.testing.assert_allclose(np.abs(_pairs(oracle.rope_rotate(row, 77, 10000.0, layout), layout)),
                               np.abs(_pairs(row, layout)), atol=1e-12)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_attention_scores_depend_on_relative_positions_only(layout):
    # the property that makes re-indexing legitimate: a key written at cache position 11 and
    # turned by (5 - 11) equals the key written at position 5, so q.k is what a fresh cache gives
    g = torch.Generator().manual_seed(3)
    q = torch.randn(64, generator=g, dtype=torch.float64)
    k = torch.randn(64, generator=g, dtype=torch.float64)
    k_old = oracle.rope_rotate(k, 11, 10000.0, layout)
    k_moved = oracle.rope_rotate(k_old, 5 - 11, 10000.0, layout)
    assert torch.allclose(k_moved, oracle.rope_rotate(k, 5, 10000.0, layout), atol=1e-12, rtol=0)
    q8 = oracle.rope_rotate(q, 8, 10000.0, layout)
    s1 = float(q8 @ k_moved)
    s2 = float(oracle.rope_rotate(q, 3, 10000.0, layout) @ k)       # relative distance 3 either way
    assert s1 == pytest.approx(s2, abs=1e-11)


def test_layouts_are_permutations_of_each_other():
    g = torch.Generator().manual_seed(4)
    row = torch.randn(32, generator=g, dtype=torch.float64)
    half = oracle.rope_rotate(row, 9, 10000.0, oracle.ROPE_HALF)
    inter = torch.empty(32, dtype=torch.float64)
    inter[0::2], inter[1::2] = row[:16], row[16:]
    out = oracle.rope_rotate(inter, 9, 10000.0, oracle.ROPE_INTERLEAVED)
    assert torch.equal(out[0::2], half[:16]) and torch.equal(out[1::2], half[16:])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_rounding_to_the_storage_type_is_round_to_nearest_even(dtype):
    g = torch.Generator().manual_seed(5)
    x = torch.cat([torch.randn(4000, generator=g) * 3, torch.randn(500, generator=g) * 1e-6,
                   torch.tensor([0.0, -0.0, 1.0, 65504.0, 6.1e-5, 5.9e-8, 1e-40, 3.3895e38])])
    want = x.to(dtype).double()                      # fp32 -> 16 bit is one correctly rounded step
    got = torch.tensor([oracle.round16(float(v), dtype == torch.bfloat16) for v in x.double()])
    ok = (got == want) | (got.isinf() & want.isinf())
    assert bool(ok.all()), x[~ok][:5]
    # exact ties go to even
    assert oracle.round16(1.0 + 2.0 ** -8, True) == 1.0 and oracle.round16(1.0 + 3 * 2.0 ** -8, True) == 1.0 + 2.0 ** -6
    assert oracle.round16(1.0 + 2.0 ** -11, False) == 1.0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_rerotating_a_plane_touches_only_moved_rows(dtype):
    g = torch.Generator().manual_seed(6)
    plane = torch.randn(12, 16, generator=g).to(dtype)
    keep = torch.tensor([0, 1, 2, 5, 6, 11])
    out = oracle.rerotate_plane(plane, keep, 10000.0, oracle.ROPE_HALF)
    assert torch.equal(out[:3], plane[:3]) and torch.equal(out[6:], plane[6:])
    for j in (3, 4, 5):
        want = oracle.rope_rotate(plane[j].double(), j - int(keep[j]), 10000.0, oracle.ROPE_HALF)
        assert torch.allclose(out[j].double(), want, rtol=2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -11,
                              atol=1e-6)
        assert not torch.equal(out[j], plane[j])
