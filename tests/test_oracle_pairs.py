"""Pins for the oracle's Token Entropy from split-vocabulary partial results (the form an
LM-head GEMM epilogue would hand over instead of the logits)."""
import math

import numpy as np
import pytest
import torch

import oracle


def tile_pairs(logits: torch.Tensor, tile: int) -> torch.Tensor:
    """Exact per-tile (max, sum exp(z - max)) in float64, rounded once to fp32."""
    T, V = logits.shape
    n = (V + tile - 1) // tile
    z = torch.full((T, n * tile), -float("inf"), dtype=torch.float64)
    z[:, :V] = logits.double()
    z = z.view(T, n, tile)
    m = z.max(dim=2).values
    s = torch.exp(z - m[:, :, None]).sum(dim=2)
    return torch.stack([m, s], dim=2).float()


@pytest.mark.parametrize("tile", [1, 7, 128, 4096])
def test_pairs_give_the_same_entropy_as_the_whole_row(tile):
    g = torch.Generator().manual_seed(tile)
    logits = (torch.randn(9, 3001, generator=g) * 3).to(torch.bfloat16).float()
    ids = torch.randint(0, 3001, (9,), generator=g, dtype=torch.int32)
    target = logits[torch.arange(9), ids.long()]
    got = oracle.score_pairs(tile_pairs(logits, tile), target, ids, 3001)
    want = oracle.score(logits, ids)
    np.testing.assert_allclose(got.numpy(), want.numpy(), rtol=0, atol=2e-6)


def test_closed_forms():
    # n tiles of W equal logits c: sum = n*W*exp(c); e = log(n*W) + c - target
    n, W, c = 10, 128, 1.5
    pairs = torch.tensor([[[c, float(W)]] * n])
    e = oracle.score_pairs(pairs, torch.tensor([c]), torch.tensor([3]), n * W)
    assert float(e) == pytest.approx(math.log(n * W), abs=1e-6)
    # a single tile is log s + m - z
    e = oracle.score_pairs(torch.tensor([[[2.0, 5.0]]]), torch.tensor([0.5]), torch.tensor([0]), 8)
    assert float(e) == pytest.approx(math.log(5.0) + 1.5, abs=1e-6)
    # ids: -1 scores 0, out of range scores 0
    e = oracle.score_pairs(torch.tensor([[[2.0, 5.0]]] * 2), torch.zeros(2), torch.tensor([-1, 8]), 8)
    assert e.tolist() == [0.0, 0.0]


def test_invariances():
    g = torch.Generator().manual_seed(5)
    pairs = torch.stack([torch.randn(4, 33, generator=g) * 4, torch.rand(4, 33, generator=g) * 100 + 1], 2)
    target = torch.randn(4, generator=g)
    ids = torch.zeros(4, dtype=torch.int32)
    base = oracle.score_pairs(pairs, target, ids, 10).double()
    perm = torch.randperm(33, generator=g)
    assert torch.allclose(oracle.score_pairs(pairs[:, perm], target, ids, 10).double(), base, atol=1e-6)
    shifted = pairs.clone()
    shifted[:, :, 0] += 8.0                                     # exact in fp32 for these magnitudes?
    shifted_t = target + 8.0
    assert torch.allclose(oracle.score_pairs(shifted, shifted_t, ids, 10).double(), base, atol=5e-6)
    # a fully masked tile (max -inf, sum 0) changes nothing
    masked = torch.cat([pairs, torch.tensor([[[-float("inf"), 0.0]]]).expand(4, 1, 2)], dim=1)
    assert torch.equal(oracle.score_pairs(masked, target, ids, 10), oracle.score_pairs(pairs, target, ids, 10))
    # rescaling a pair consistently, (m, s) -> (m + ln 2, s / 2), keeps its contribution
    rs = pairs.double().clone()
    rs[:, 5, 0] += math.log(2.0)
    rs[:, 5, 1] /= 2.0
    assert torch.allclose(oracle.score_pairs(rs.float(), target, ids, 10).double(), base, atol=1e-6)


# ---- one rank's column range (vocabulary-parallel LM head) ---------------------------------

@pytest.mark.parametrize("cuts", [[0, 3001], [0, 1, 3001], [0, 1500, 3001], [0, 7, 7, 2999, 3000, 3001],
                                  [0, 1024, 2048, 3001], [0, 0, 3001, 3001]])
def test_uneven_column_ranges_give_the_same_entropy_as_the_whole_row(cuts):
    # any cutting of the vocabulary into contiguous ranges - uneven, single-column, empty - must
    # reproduce the whole-row definition once the ranges' pairs are combined
    g = torch.Generator().manual_seed(len(cuts))
    for dtype in (torch.float32, torch.bfloat16):
        logits = (torch.randn(7, 3001, generator=g) * 3).to(dtype)
        logits[2, 100:900] = -float("inf")                      # a stretch of masked columns
        ids = torch.randint(0, 3001, (7,), generator=g, dtype=torch.int32)
        ids[2] = 950
        ids[3] = -1
        parts = [oracle.range_pairs(logits, ids, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
        pairs = torch.stack([p for p, _ in parts], dim=1)       # [T, ranks, 2]
        target = torch.stack([t for _, t in parts]).sum(dim=0)  # only the owning range is non-zero
        assert torch.equal(target[ids >= 0], logits.float()[torch.arange(7), ids.long().clamp(min=0)][ids >= 0])
        got = oracle.score_pairs(pairs, target, ids, 3001)
        want = oracle.score(logits, ids)
        np.testing.assert_allclose(got.numpy(), want.numpy(), rtol=0, atol=2e-6)
        assert float(got[3]) == 0.0


def test_range_pair_closed_forms():
    # n equal logits c in the range: (c, n); a fully masked or empty range: (0, 0)
    row = torch.full((1, 64), 1.25)
    row[0, 40:] = -float("inf")
    ids = torch.tensor([5], dtype=torch.int32)
    p, t = oracle.range_pairs(row, ids, 0, 32)
    assert p.tolist() == [[1.25, 32.0]] and t.tolist() == [1.25]
    p, t = oracle.range_pairs(row, ids, 32, 64)                 # 8 live columns, 24 masked
    assert p.tolist() == [[1.25, 8.0]] and t.tolist() == [0.0]
    p, t = oracle.range_pairs(row, ids, 40, 64)
    assert p.tolist() == [[0.0, 0.0]]
    p, t = oracle.range_pairs(row, ids, 10, 10)
    assert p.tolist() == [[0.0, 0.0]] and t.tolist() == [0.0]
    # the maximum is the range's own, whatever the rest of the row holds
    row = torch.cat([torch.full((1, 32), 5.0), torch.full((1, 32), 1.25)], dim=1)
    p, _ = oracle.range_pairs(row, ids, 32, 64)
    assert p.tolist() == [[1.25, 32.0]]
    # two columns (0, ln 3): max ln 3, sum 1 + 1/3
    row = torch.tensor([[0.0, math.log(3.0)]])
    p, _ = oracle.range_pairs(row, torch.tensor([0], dtype=torch.int32), 0, 2)
    assert float(p[0, 0]) == pytest.approx(math.log(3.0), abs=1e-7)
    assert float(p[0, 1]) == pytest.approx(4.0 / 3.0, abs=1e-7)
