"""Pins for the oracle's round composition (Algorithm 1: append, decay, evict-if-over)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2405_12528_b200 import workloads as wl


def _stream(capacity=64, n_sink=2, n_recent=4, budget=16, threshold=None, eta=0.9, planes=0, dim=8):
    k = v = None
    if planes:
        k = torch.zeros(planes, capacity, dim, dtype=torch.float16)
        v = torch.zeros(planes, capacity, dim, dtype=torch.float16)
    return oracle.Stream(capacity, n_sink, n_recent, budget, threshold or budget, eta, k, v)


def test_each_score_is_decayed_once_per_round_from_its_first_round_on():
    # Algorithm 1 appends the round's scores and then multiplies the whole cache
    s = _stream(capacity=40, budget=36, eta=0.7)
    eta = np.float32(0.7)
    first = {}
    g = torch.Generator().manual_seed(0)
    for r in range(6):
        new = torch.rand(5, generator=g) + 1
        base = int(s.next_serial.value)
        s.step(new)
        for t in range(5):
            first[base + t] = (r, np.float32(new[t]))
        for j in range(s.live_len):
            r0, val = first[int(s.serial[j])]
            for _ in range(r - r0 + 1):
                val = np.float32(val * eta)
            assert np.float32(s.E[j]) == val
    assert s.live_len == 30 and s.keep.tolist() == list(range(30))


def test_eviction_happens_only_above_the_threshold_and_restores_the_budget():
    s = _stream(capacity=64, budget=16, threshold=24, eta=1.0)
    lens = []
    for r in range(8):
        s.step(torch.arange(6, dtype=torch.float32) + r)
        lens.append(s.live_len)
    # 6,12,18,24 (== threshold: kept), 30 -> 16, 22, 28 -> 16, 22
    assert lens == [6, 12, 18, 24, 16, 22, 16, 22]


def test_rows_follow_their_tokens_through_compaction():
    w = wl.WORKLOADS["tiny"].scaled(n_layers=1, n_kv_heads=3, head_dim=8, capacity=48, budget=20,
                                    n_sink=2, n_recent=5, new_tokens=9)
    planes = w.planes_per_stream
    s = oracle.Stream(w.capacity, w.n_sink, w.n_recent, w.budget, w.budget, 0.8,
                      torch.zeros(planes, w.capacity, w.head_dim, dtype=torch.float16),
                      torch.zeros(planes, w.capacity, w.head_dim, dtype=torch.float16))
    g = torch.Generator().manual_seed(1)
    for r in range(7):
        l, T = s.live_len, w.new_tokens
        serials = torch.arange(int(s.next_serial.value), int(s.next_serial.value) + T)
        s.k[:, l:l + T] = wl.make_kv_rows(w, 0, "k", 0, serials)
        s.v[:, l:l + T] = wl.make_kv_rows(w, 0, "v", 0, serials)
        s.step(torch.rand(T, generator=g) * 10)
        live = s.serial[:s.live_len]
        assert (live[1:] > live[:-1]).all()                       # text order is preserved
        assert torch.equal(s.k[:, :s.live_len], wl.make_kv_rows(w, 0, "k", 0, live))
        assert torch.equal(s.v[:, :s.live_len], wl.make_kv_rows(w, 0, "v", 0, live))
        assert live[:w.n_sink].tolist() == list(range(w.n_sink))  # the first tokens never leave
        if r >= 2:
            assert s.live_len == w.budget
            newest = int(s.next_serial.value)
            assert live[-w.n_recent:].tolist() == list(range(newest - w.n_recent, newest))


def test_forgetting_horizon_with_decay_below_one():
    # With new scores in [e_min, e_max] and eta < 1, a middle token older than
    # ceil(ln(e_min / e_max) / ln(eta)) rounds scores below every newer one and is evicted
    # once enough newer candidates exist (the decay study of Appendix B: eta < 1 forgets).
    e_min, e_max, eta, T = 2.0, 12.0, 0.7, 10
    horizon = math.ceil(math.log(e_min / e_max) / math.log(eta))
    s = _stream(capacity=100, n_sink=4, n_recent=0, budget=4 + 30, eta=eta)
    g = torch.Generator().manual_seed(2)
    born = {}
    for r in range(40):
        base = int(s.next_serial.value)
        s.step(e_min + (e_max - e_min) * torch.rand(T, generator=g))
        for t in range(T):
            born[base + t] = r
        ages = [r - born[int(x)] for x in s.serial[4:s.live_len]]
        if r > horizon + 4:
            # k = 30 = three rounds of candidates (ages 0..2), and age a loses to every age
            # <= a - horizon: nothing older than horizon + 1 rounds survives
            assert max(ages) <= horizon + 1
    # with eta = 1 the best old tokens stay forever ("rigid memory", Section 3.3)
    s = _stream(capacity=100, n_sink=4, n_recent=0, budget=4 + 30, eta=1.0)
    first = torch.full((T,), 50.0)
    s.step(torch.cat([torch.zeros(4), first]))
    for r in range(40):
        s.step(e_min + (e_max - e_min) * torch.rand(T, generator=g))
    assert set(range(4, 4 + T)) <= set(s.serial[:s.live_len].tolist())


def test_round_that_does_not_fit_is_refused_and_empty_round_only_decays():
    s = _stream(capacity=20, budget=16, eta=0.5)
    s.step(torch.ones(10))
    with pytest.raises(ValueError):
        s.step(torch.ones(11))
    assert s.live_len == 10 and s.E[:10].tolist() == [0.5] * 10
    s.step(torch.ones(0))
    assert s.live_len == 10 and s.E[:10].tolist() == [0.25] * 10


def test_more_new_tokens_than_budget_evicts_inside_the_round():
    # the tiny workload: 512 new tokens into a budget of 256
    w = wl.WORKLOADS["tiny"]
    s = oracle.Stream(w.capacity, w.n_sink, w.n_recent, w.budget, w.budget, w.decay)
    e = wl.random_scores(7, w.new_tokens)
    keep = s.step(e)
    assert s.live_len == w.budget and len(keep) == w.budget
    assert keep[:4].tolist() == [0, 1, 2, 3] and keep[-64:].tolist() == list(range(448, 512))
    mid = keep[4:-64].long()
    dec = (e.numpy() * np.float32(w.decay)).astype(np.float32)
    cut = np.sort(dec[4:448])[::-1][w.budget - 68 - 1]
    assert (dec[mid.numpy()] >= cut).all()


def _read_trace(path):
    head, rounds = {}, []
    for line in open(path):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "round":
            rounds.append({"new": [float(x) for x in f[1:]]})
        elif f[0] in ("kept", "tokens"):
            rounds[-1][f[0]] = [int(x) for x in f[1:]]
        elif f[0] == "scores":
            rounds[-1]["scores"] = [float(x) for x in f[1:]]
        else:
            head[f[0]] = float(f[1])
    return head, rounds


def test_rounds_worked_by_hand_from_algorithm_1(golden_dir):
    # seven rounds of Algorithm 1 followed on paper (exact binary scores, decay 0.5): pins the
    # order append -> decay -> evict, the three index sets, the tie rule, the compaction of
    # scores, tags and rows, and a round without new tokens
    head, rounds = _read_trace(f"{golden_dir}/algorithm1_hand_trace.txt")
    cap, dim = 8, 4
    s = oracle.Stream(cap, int(head["n_sink"]), int(head["n_recent"]), int(head["budget"]),
                      int(head["threshold"]), head["decay"],
                      torch.zeros(2, cap, dim, dtype=torch.float16), torch.zeros(2, cap, dim, dtype=torch.float16))
    assert len(rounds) == 7
    for r in rounds:
        T, l, first = len(r["new"]), s.live_len, int(s.next_serial.value)
        for t in range(T):                       # the round's rows carry the token's number
            s.k[:, l + t] = first + t
            s.v[:, l + t] = -(first + t)
        keep = s.step(torch.tensor(r["new"], dtype=torch.float32))
        n = s.live_len
        assert keep.tolist() == r["kept"]
        assert s.serial[:n].tolist() == r["tokens"]
        assert s.E[:n].tolist() == r["scores"]
        for p in range(2):
            assert s.k[p, :n, 0].tolist() == [float(x) for x in r["tokens"]]
            assert s.v[p, :n, dim - 1].tolist() == [-float(x) for x in r["tokens"]]
