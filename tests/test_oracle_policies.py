"""Pins for the oracle's versions of the paper's comparison policies (Section 4.1.1)."""
import numpy as np
import pytest
import torch

import oracle


def test_philox_known_answers(golden_dir):
    import os
    n = 0
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(t, 16) for t in line.split()]
            assert oracle.philox4x32_10(w[0:4], w[4:6]) == w[6:10]
            n += 1
    assert n == 3


def test_stream_policy_is_sinks_plus_most_recent():
    assert oracle.keep_policy(oracle.STREAM, 100, 4, 0, 32).tolist() == [0, 1, 2, 3] + list(range(72, 100))
    assert oracle.keep_policy(oracle.STREAM, 20, 4, 0, 32).tolist() == list(range(20))
    # identical to the entropy policy with no top-k slots (k = 0)
    E = torch.rand(100)
    assert oracle.keep_policy(oracle.STREAM, 100, 4, 0, 32).tolist() == oracle.select(E, 100, 4, 28, 32).tolist()


def test_interval_policy_hand_computed():
    # history 100, cache 32: interval = 3; sinks 0..3 then 4, 7, 10, ... until 32 slots are used
    keep = oracle.keep_policy(oracle.INTERVAL, 100, 4, 0, 32).tolist()
    assert keep == [0, 1, 2, 3] + [4 + 3 * j for j in range(28)]
    # interval 1 (history < 2 x cache): the oldest tokens fill the cache
    assert oracle.keep_policy(oracle.INTERVAL, 50, 4, 0, 32).tolist() == list(range(32))
    # with a recent window the last slots stay as well
    keep = oracle.keep_policy(oracle.INTERVAL, 100, 4, 8, 32).tolist()
    assert keep == [0, 1, 2, 3] + [4 + 3 * j for j in range(20)] + list(range(92, 100))
    assert oracle.keep_policy(oracle.INTERVAL, 30, 4, 0, 32).tolist() == list(range(30))


def test_random_policy_invariants_and_uniformity():
    l, n_sink, n_recent, budget = 200, 4, 6, 60
    k, n_mid = budget - n_sink - n_recent, l - n_sink - n_recent
    counts = np.zeros(l)
    seen = set()
    trials = 600
    for seed in range(trials):
        keep = oracle.keep_policy(oracle.RANDOM, l, n_sink, n_recent, budget, seed=seed, stream=1, rnd=2)
        kl = keep.tolist()
        assert len(kl) == budget and kl == sorted(set(kl))
        assert kl[:n_sink] == list(range(n_sink)) and kl[-n_recent:] == list(range(l - n_recent, l))
        counts[kl] += 1
        seen.add(tuple(kl))
    assert len(seen) == trials                                   # seeds give different subsets
    p = k / n_mid
    mid = counts[n_sink:l - n_recent] / trials
    sigma = (p * (1 - p) / trials) ** 0.5
    assert np.abs(mid - p).max() < 5 * sigma                     # every middle slot kept with prob k/n
    assert abs(mid.mean() - p) < 1e-12
    # stream and round are part of the counter
    a = oracle.keep_policy(oracle.RANDOM, l, n_sink, n_recent, budget, seed=7, stream=0, rnd=0)
    assert not torch.equal(a, oracle.keep_policy(oracle.RANDOM, l, n_sink, n_recent, budget, seed=7, stream=1, rnd=0))
    assert not torch.equal(a, oracle.keep_policy(oracle.RANDOM, l, n_sink, n_recent, budget, seed=7, stream=0, rnd=1))
    assert torch.equal(a, oracle.keep_policy(oracle.RANDOM, l, n_sink, n_recent, budget, seed=7, stream=0, rnd=0))
    assert oracle.keep_policy(oracle.RANDOM, 40, 4, 6, 60).tolist() == list(range(40))
