"""Pins for the oracle's decay, selection rule and row gather (Sections 3.1, 3.3, Algorithm 1)."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st

import oracle


# ----------------------------------------------------------------------------- decay

def test_decay_ratio_one_is_a_bitwise_identity():
    # the Grocery Shopping runs use a decay ratio of 1 (Section 4.2.2)
    E = torch.tensor([0.0, -0.0, 1.17549435e-38, 1e-45, 3.3, 65504.0, float("inf")])
    before = E.view(torch.int32).clone()
    oracle.decay(E, E.numel(), 1.0)
    assert torch.equal(E.view(torch.int32), before)


@pytest.mark.parametrize("eta", [0.5, 0.6, 0.7, 0.8, 0.9])
def test_decay_is_one_fp32_multiply_per_round(eta):
    g = torch.Generator().manual_seed(0)
    E0 = torch.rand(257, generator=g) * 15
    E = E0.clone()
    ref = E0.numpy().copy()
    eta32 = np.float32(eta)
    rounds = 40
    for _ in range(rounds):
        oracle.decay(E, 257, eta)
        ref = (ref * eta32).astype(np.float32)         # numpy's correctly rounded fp32 product
    np.testing.assert_array_equal(E.numpy(), ref)
    closed = E0.double().numpy() * float(eta32) ** rounds
    ulp = np.spacing(np.abs(closed).astype(np.float32)).astype(np.float64)
    assert (np.abs(E.double().numpy() - closed) <= rounds * ulp).all()


def test_decay_only_touches_the_live_prefix():
    E = torch.ones(10)
    oracle.decay(E, 6, 0.5)
    assert E.tolist() == [0.5] * 6 + [1.0] * 4


def test_decay_keeps_denormals_and_underflows_to_zero_exactly():
    E = torch.ones(1)
    for r in range(1, 161):
        oracle.decay(E, 1, 0.5)
        want = math.ldexp(1.0, -r) if r <= 149 else 0.0     # 2**-150 ties to even -> 0
        assert float(E[0]) == want, r


# ----------------------------------------------------------------------------- order key

def test_order_key_is_monotone_in_the_score():
    vals = [-float("inf"), -3.5, -1e-45, -0.0, 0.0, 1e-45, 1.17549435e-38, 0.1, 1.0, 1.0000001,
            7.25, 3.4e38, float("inf")]
    keys = [oracle.order_key(v) for v in vals]
    assert keys == sorted(keys) and len(set(keys)) == len(keys)
    g = np.random.default_rng(0)
    x = g.standard_normal(2000).astype(np.float32) * np.float32(50)
    k = np.array([oracle.order_key(float(v)) for v in x], dtype=np.uint64)
    order = np.argsort(x, kind="stable")
    assert (np.diff(k[order].astype(np.int64)) >= 0).all()
    assert ((x[:, None] < x[None, :]) == (k[:, None] < k[None, :])).all()


# ----------------------------------------------------------------------------- selection

def _read_example(golden_dir):
    vals = {}
    with open(os.path.join(golden_dir, "paper_cache_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            name, *rest = line.split()
            vals[name] = [int(t) for t in rest]
    return vals


def test_paper_printed_cache_example(golden_dir):
    ex = _read_example(golden_dir)
    l, = ex["live_len"]
    n_sink, = ex["n_sink"]
    n_recent, = ex["n_recent"]
    budget, = ex["budget"]
    E = torch.full((l,), 1.0)
    E[5], E[7] = 9.0, 6.5            # the two middle tokens worth remembering
    E[0], E[12] = 0.01, 0.02         # sinks / recent stay however low they score
    E[4], E[9] = 5.0, 6.0            # good, but not good enough
    keep = oracle.select(E, l, n_sink, n_recent, budget)
    assert keep.tolist() == ex["kept"]
    # positions are assigned by order inside the cache
    serial = torch.arange(l)
    assert oracle.gather_rows(serial, keep).tolist() == ex["kept"]
    assert list(range(len(keep))) == ex["positions"]


def test_no_top_k_slots_reduces_to_sinks_plus_recent_window():
    # StreamLLM (Section 3.1): Id_sink U Id_recent
    g = torch.Generator().manual_seed(1)
    for l, n_sink, n_recent in [(100, 4, 28), (33, 4, 28), (50, 0, 10), (50, 6, 0)]:
        E = torch.rand(l, generator=g)
        keep = oracle.select(E, l, n_sink, n_recent, n_sink + n_recent)
        assert keep.tolist() == list(range(n_sink)) + list(range(l - n_recent, l))


def test_under_threshold_nothing_is_evicted():
    E = torch.rand(20)
    assert oracle.select(E, 20, 4, 4, 20).tolist() == list(range(20))
    assert oracle.select(E, 20, 4, 4, 12, threshold=20).tolist() == list(range(20))
    assert oracle.select(E, 0, 4, 4, 12).tolist() == []
    assert oracle.select(E, 3, 4, 4, 12).tolist() == [0, 1, 2]
    assert len(oracle.select(E, 20, 4, 4, 12, threshold=19)) == 12


def test_all_equal_scores_keep_the_oldest_candidates():
    E = torch.full((40,), 2.5)
    keep = oracle.select(E, 40, 4, 6, 20)
    assert keep.tolist() == list(range(4)) + list(range(4, 14)) + list(range(34, 40))
    # decayed-to-zero history behaves the same way
    E = torch.zeros(40)
    assert oracle.select(E, 40, 4, 6, 20).tolist() == keep.tolist()


def _brute_force(E, l, n_sink, n_recent, budget):
    """Best k-subset of the middle by exhaustive search: compare subsets by their
    members sorted best-first, a member being better if it scores higher or, on a
    tie, sits in the lower slot."""
    lo, hi, k = n_sink, l - n_recent, budget - n_sink - n_recent
    best, best_rank = None, None
    for sub in itertools.combinations(range(lo, hi), k):
        rank = sorted(((-float(E[i]), i) for i in sub))
        if best is None or rank < best_rank:
            best, best_rank = sub, rank
    return sorted(list(range(lo)) + list(best) + list(range(hi, l)))


@pytest.mark.parametrize("seed", range(12))
def test_selection_against_exhaustive_search(seed):
    g = np.random.default_rng(seed)
    l = int(g.integers(6, 13))
    n_sink = int(g.integers(0, 3))
    n_recent = int(g.integers(0, 3))
    k = int(g.integers(0, l - n_sink - n_recent))
    budget = n_sink + n_recent + k
    if seed % 2:
        E = torch.tensor(g.integers(0, 4, l).astype(np.float32) * 0.5)      # many ties
    else:
        E = torch.tensor(g.random(l).astype(np.float32))
    assert budget < l
    got = oracle.select(E, l, n_sink, n_recent, budget).tolist()
    assert got == _brute_force(E, l, n_sink, n_recent, budget)


@settings(max_examples=150, deadline=None)
@given(st.integers(0, 2**31 - 1), st.integers(1, 300), st.integers(0, 8), st.integers(0, 40),
       st.integers(0, 120), st.integers(0, 30), st.booleans())
def test_selection_invariants(seed, l, n_sink, n_recent, k, slack, ties):
    budget = n_sink + n_recent + k
    threshold = budget + slack
    g = torch.Generator().manual_seed(seed)
    E = torch.rand(l, generator=g) * 10
    if ties:
        E = torch.round(E)
    keep = oracle.select(E, l, n_sink, n_recent, budget, threshold).tolist()
    if l <= threshold:
        assert keep == list(range(l))
        return
    assert len(keep) == budget                                  # retained count equals budget
    assert keep == sorted(set(keep))                            # ascending, no repeats
    assert keep[:n_sink] == list(range(n_sink))                 # sinks kept
    assert keep[budget - n_recent:] == list(range(l - n_recent, l))   # recent window kept
    mid = set(keep[n_sink:budget - n_recent])
    assert all(n_sink <= i < l - n_recent for i in mid)
    out = [i for i in range(n_sink, l - n_recent) if i not in mid]
    if mid and out:
        worst_in = min((float(E[i]), -i) for i in mid)
        best_out = max((float(E[i]), -i) for i in out)
        assert worst_in > best_out                              # nobody evicted outranks a kept one


def test_inconsistent_parameters_are_rejected():
    E = torch.rand(10)
    with pytest.raises(ValueError):
        oracle.select(E, 10, 4, 4, 6)
    with pytest.raises(ValueError):
        oracle.select(E, 10, 2, 2, 8, threshold=6)


# ----------------------------------------------------------------------------- gather

def test_gather_is_x_of_id():
    g = torch.Generator().manual_seed(3)
    src = torch.randn(50, 16, generator=g).to(torch.bfloat16)
    keep = torch.tensor([0, 1, 5, 6, 7, 30, 49], dtype=torch.int32)
    assert torch.equal(oracle.gather_rows(src, keep), src[keep.long()])
    ident = torch.arange(50, dtype=torch.int32)
    assert torch.equal(oracle.gather_rows(src, ident), src)
    assert oracle.gather_rows(src, keep[:0]).shape == (0, 16)
