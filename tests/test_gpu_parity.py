"""CUDA path against the CPU oracle, through the C ABI, on the same seeded inputs.

Scores: within max(1e-5, 1e-4*|e|).  Keep lists, compacted scores, tags and K/V: bit exact
(the oracle's selection consumes the GPU's scores, so both sides rank identical numbers).
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import DeviceState, assert_entropy_close, oracle_twin
from paper_2405_12528_b200 import binding as B
from paper_2405_12528_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _score_cfg(T, V, dtype, stride=None, n_streams=1):
    return B.make_config(n_streams, 1, 1, 8, 64, 16, 2, 2, T, V, dtype, torch.bfloat16,
                         logits_row_stride=stride)


# ------------------------------------------------------------------------------- scoring

def test_score_tiny_workload_fp32():
    w = wl.WORKLOADS["tiny"]
    st = DeviceState(w, with_kv=False)
    st.fill_round(0)
    out = torch.full((w.new_tokens,), -1.0, device=DEV)
    B.sirllm_score(st.cfg, st.logits, st.token_ids, None, out, st.ws)
    want = oracle.score(st.logits.cpu(), st.token_ids.cpu())
    assert_entropy_close(out, want)
    assert B.sirllm_status(st.ws) == 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("V,stride", [(1, None), (2, None), (7, 9), (33, None), (4095, 4099),
                                      (4096, None), (8193, 8200), (32000, None), (50257, 50257)])
def test_score_ragged_vocabularies_and_strides(dtype, V, stride):
    # odd V and odd strides put rows off the 16-byte grid: ragged head and tail per row;
    # V > 4096 (bf16) / 2048 (fp32) spans several segments
    T = 19
    stride = V if stride is None else stride
    g = torch.Generator().manual_seed(V)
    buf = (torch.randn(T, stride, generator=g) * 3).to(dtype)
    ids = torch.randint(0, V, (T,), generator=g, dtype=torch.int32)
    cfg = _score_cfg(T, V, dtype, stride)
    ws = B.new_workspace(cfg)
    out = torch.zeros(T, device=DEV)
    d_buf = buf.to(DEV)
    B.sirllm_score(cfg, d_buf[:, :V] if stride != V else d_buf, ids.to(DEV), None, out, ws)
    assert_entropy_close(out, oracle.score(buf[:, :V], ids))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_score_rows_of_a_million_logits(dtype):
    # a row far wider than any model's vocabulary: dozens of CTAs reduce one row and the last one
    # to arrive combines their pairs; odd width, odd stride, targets in the first, a middle and
    # the last column, and one id that has no prediction
    T, V, stride = 5, 1_000_003, 1_000_011
    g = torch.Generator().manual_seed(5)
    buf = (torch.randn(T, stride, generator=g) * 2.5).to(dtype)
    ids = torch.tensor([0, V // 2, V - 1, -1, 12345], dtype=torch.int32)
    cfg = _score_cfg(T, V, dtype, stride)
    ws = B.new_workspace(cfg)
    out = torch.full((T,), -1.0, device=DEV)
    B.sirllm_score(cfg, buf.to(DEV)[:, :V], ids.to(DEV), None, out, ws)
    assert_entropy_close(out, oracle.score(buf[:, :V], ids))
    assert float(out[3]) == 0.0 and B.sirllm_status(ws) == 0


def test_score_closed_forms_on_device():
    import math
    V = 32000
    cfg = _score_cfg(3, V, torch.float32)
    ws = B.new_workspace(cfg)
    z = torch.zeros(3, V)
    z[1, 77] = 80.0
    z[2] = -5.0
    z[2, 0] = float("-inf")              # a masked column
    ids = torch.tensor([5, 77, 9], dtype=torch.int32)
    out = torch.zeros(3, device=DEV)
    B.sirllm_score(cfg, z.to(DEV), ids.to(DEV), None, out, ws)
    out = out.cpu()
    assert abs(float(out[0]) - math.log(V)) < 1e-5
    assert float(out[1]) == 0.0
    assert abs(float(out[2]) - math.log(V - 1)) < 1e-5


def test_score_special_ids_ragged_streams_and_status():
    S, M, V = 3, 8, 1000
    cfg = _score_cfg(M, V, torch.bfloat16, n_streams=S)
    ws = B.new_workspace(cfg)
    g = torch.Generator().manual_seed(0)
    logits = (torch.randn(S * M, V, generator=g) * 2).to(torch.bfloat16)
    ids = torch.randint(0, V, (S * M,), generator=g, dtype=torch.int32)
    ids[0], ids[9], ids[10] = -1, V, -5
    n_new = torch.tensor([8, 3, 0], dtype=torch.int32)
    out = torch.full((S * M,), -7.0, device=DEV)
    B.sirllm_score(cfg, logits.to(DEV), ids.to(DEV), n_new.to(DEV), out, ws)
    out = out.cpu()
    want = oracle.score(logits, ids)
    live = torch.zeros(S * M, dtype=torch.bool)
    for s in range(S):
        live[s * M:s * M + int(n_new[s])] = True
    assert_entropy_close(out[live], want[live])
    assert (out[~live] == -7.0).all()                    # rows beyond n_new are not touched
    assert out[0] == 0.0 and out[9] == 0.0 and out[10] == 0.0
    assert B.sirllm_status(ws, clear=True) == B.STATUS_TOKEN_RANGE
    assert B.sirllm_status(ws) == 0


# ------------------------------------------------------------------------------- selection

def _select_case(l_list, n_sink, n_recent, budget, threshold, cap, seed, quantise, decay, compact):
    S = len(l_list)
    cfg = B.make_config(S, 1, 1, 8, cap, budget, n_sink, n_recent, 0, 16, torch.float32,
                        torch.bfloat16, threshold=threshold)
    ws = B.new_workspace(cfg)
    E = torch.zeros(S, cap)
    serial = torch.full((S, cap), -1, dtype=torch.int64)
    for s, l in enumerate(l_list):
        E[s, :l] = wl.random_scores(seed + s, l, quantise=quantise)
        serial[s, :l] = torch.arange(l) * 3 + s
    dE, dser = E.to(DEV), serial.to(DEV)
    dlen = torch.tensor(l_list, dtype=torch.int32, device=DEV)
    ddec = torch.tensor(decay, dtype=torch.float32, device=DEV)
    keep = torch.full((S, threshold), -1, dtype=torch.int32, device=DEV)
    nk = torch.zeros(S, dtype=torch.int32, device=DEV)
    B.sirllm_decay_select(cfg, dE, dser, dlen, ddec, keep, nk, compact, ws)
    assert B.sirllm_status(ws) == 0
    for s, l in enumerate(l_list):
        Es = E[s].clone()
        oracle.decay(Es, l, decay[s])
        want = oracle.select(Es, l, n_sink, n_recent, budget, threshold)
        n = int(nk[s])
        assert n == len(want)
        assert torch.equal(keep[s, :n].cpu(), want)
        if compact:
            assert int(dlen[s]) == n
            assert torch.equal(dE[s, :n].cpu().view(torch.int32), Es[want.long()].view(torch.int32))
            assert torch.equal(dser[s, :n].cpu(), serial[s][want.long()])
        else:
            assert int(dlen[s]) == l
            assert torch.equal(dE[s, :l].cpu().view(torch.int32), Es[:l].view(torch.int32))
            assert torch.equal(dser[s].cpu(), serial[s])


@pytest.mark.parametrize("compact", [False, True])
@pytest.mark.parametrize("quantise", [0, 5])
def test_select_matches_oracle(compact, quantise):
    _select_case([5000, 3000, 2049, 2048, 100, 0], 4, 256, 2048, 2048, 5120, 1, quantise,
                 [0.9, 0.5, 1.0, 0.7, 0.8, 0.9], compact)


def test_select_paper_shaped_rows_no_recent_window():
    # Tables 1-3: 4 sinks + 508 (1020) entropy slots, no recent window
    _select_case([632, 513], 4, 0, 512, 512, 640, 3, 0, [0.7, 0.5], True)
    _select_case([1078], 4, 0, 1024, 1024, 1152, 4, 7, [0.8], True)


def test_select_degenerate_shapes():
    _select_case([300], 4, 28, 32, 32, 512, 5, 0, [0.9], True)       # k = 0: StreamLLM
    _select_case([300], 0, 32, 32, 32, 512, 6, 0, [0.9], True)       # sliding window
    _select_case([300], 0, 0, 32, 32, 512, 7, 3, [0.9], True)        # pure top-k with ties
    _select_case([300, 41], 4, 4, 40, 200, 512, 8, 0, [0.9, 0.9], True)   # threshold > budget
    _select_case([33], 4, 4, 32, 32, 64, 9, 2, [1.0], True)          # evict exactly one


def test_select_largest_capacity_and_all_equal_scores():
    cap = B.MAX_CAPACITY
    _select_case([cap], 4, 1024, 8192, 8192, cap, 10, 0, [0.9], True)
    S, l = 1, 4000
    cfg = B.make_config(S, 1, 1, 8, 4096, 1000, 4, 96, 0, 16, torch.float32, torch.bfloat16)
    ws = B.new_workspace(cfg)
    E = torch.full((1, 4096), 2.5, device=DEV)
    keep = torch.zeros(1, 1000, dtype=torch.int32, device=DEV)
    nk = torch.zeros(1, dtype=torch.int32, device=DEV)
    dlen = torch.tensor([l], dtype=torch.int32, device=DEV)
    B.sirllm_decay_select(cfg, E, None, dlen, torch.tensor([0.5], device=DEV), keep, nk, 0, ws)
    assert keep[0].cpu().tolist() == list(range(904)) + list(range(l - 96, l))


def test_select_special_values_follow_the_bit_pattern_order():
    vals = torch.tensor([0.0, -0.0, 1e-45, -1e-45, float("inf"), -float("inf"), 1.0, -1.0,
                         1.17549435e-38, 3.0, 3.0, 2.0, 0.0, -0.0, 5e-324, 7.0])
    l = vals.numel()
    cfg = B.make_config(1, 1, 1, 8, 32, 6, 0, 0, 0, 16, torch.float32, torch.bfloat16)
    ws = B.new_workspace(cfg)
    E = torch.zeros(1, 32)
    E[0, :l] = vals
    dE = E.to(DEV)
    keep = torch.zeros(1, 6, dtype=torch.int32, device=DEV)
    nk = torch.zeros(1, dtype=torch.int32, device=DEV)
    for budget in (6, 11, 13):
        cfg = B.make_config(1, 1, 1, 8, 32, budget, 0, 0, 0, 16, torch.float32, torch.bfloat16)
        keep = torch.zeros(1, budget, dtype=torch.int32, device=DEV)
        d = E.to(DEV)
        B.sirllm_decay_select(cfg, d, None, torch.tensor([l], dtype=torch.int32, device=DEV),
                              torch.tensor([1.0], device=DEV), keep, nk, 0, ws)
        want = oracle.select(E[0].clone(), l, 0, 0, budget)
        assert torch.equal(keep[0].cpu(), want)


# ------------------------------------------------------------------------------- compaction

def _compact_case(S, planes, cap, D, n_list, in_place, seed, dtype=torch.bfloat16):
    thr = max(n_list + [1])
    cfg = B.make_config(S, planes, 1, D, cap, thr, 0, 0, 0, 16, torch.float32, dtype)
    ws = B.new_workspace(cfg)
    g = torch.Generator().manual_seed(seed)
    k = torch.randn(S, planes, cap, D, generator=g).to(dtype)
    v = torch.randn(S, planes, cap, D, generator=g).to(dtype)
    keep = torch.full((S, thr), -1, dtype=torch.int32)
    for s, n in enumerate(n_list):
        keep[s, :n] = torch.sort(torch.randperm(cap, generator=g)[:n]).values.to(torch.int32)
    dk, dv = k.to(DEV), v.to(DEV)
    dkeep, dn = keep.to(DEV), torch.tensor(n_list, dtype=torch.int32, device=DEV)
    if in_place:
        B.sirllm_compact_kv(cfg, dk, dv, dk, dv, dkeep, dn, ws)
        ok, ov = dk, dv
    else:
        ok = torch.full_like(dk, 9.0)
        ov = torch.full_like(dv, 9.0)
        B.sirllm_compact_kv(cfg, dk, dv, ok, ov, dkeep, dn, ws)
        assert torch.equal(dk.cpu(), k) and torch.equal(dv.cpu(), v)      # sources untouched
    assert B.sirllm_status(ws) == 0
    ok, ov = ok.cpu(), ov.cpu()
    for s, n in enumerate(n_list):
        for p in range(planes):
            assert torch.equal(ok[s, p, :n], oracle.gather_rows(k[s, p], keep[s, :n]))
            assert torch.equal(ov[s, p, :n], oracle.gather_rows(v[s, p], keep[s, :n]))
            if not in_place:
                assert (ok[s, p, n:] == 9.0).all()                        # nothing written past n_keep
            else:
                # slots never used as a destination keep their old rows
                assert torch.equal(ok[s, p, n:], k[s, p, n:])


@pytest.mark.parametrize("in_place", [True, False])
def test_compact_matches_gather(in_place):
    _compact_case(2, 5, 300, 128, [200, 37], in_place, 0)
    _compact_case(1, 3, 1000, 64, [999], in_place, 1, torch.float16)       # ragged last chunk
    _compact_case(3, 2, 64, 8, [0, 1, 64], in_place, 2)                    # empty, single, full
    _compact_case(1, 700, 96, 128, [50], in_place, 3)                      # more planes than workers
    _compact_case(1, 6, 400, 256, [333], in_place, 4)                      # 512-byte rows
    _compact_case(2, 3, 200, 512, [150, 199], in_place, 5)                 # 1 KB rows: the largest


@pytest.mark.parametrize("in_place", [True, False])
def test_compact_row_widths_through_the_persistent_gather(in_place):
    # jobs of tens of MB (the ring kernel, not the two-phase one) at the narrowest row, an odd
    # multiple of 16 bytes, and the widest row (one worker per CTA)
    _compact_case(4, 512, 600, 8, [500, 600, 1, 77], in_place, 6)           # 16-byte rows
    _compact_case(2, 256, 500, 40, [400, 123], in_place, 7, torch.float16)  # 80-byte rows
    _compact_case(1, 64, 300, 512, [250], in_place, 8)                      # 1 KB rows


def test_compact_identity_list_moves_nothing_and_bad_lists_are_refused():
    cfg = B.make_config(2, 2, 1, 16, 40, 20, 0, 0, 0, 16, torch.float32, torch.bfloat16)
    ws = B.new_workspace(cfg)
    k = torch.randn(2, 2, 40, 16).to(torch.bfloat16)
    dk = k.to(DEV)
    keep = torch.stack([torch.arange(20), torch.arange(20)]).to(torch.int32)
    keep[1, 5], keep[1, 6] = 9, 8                              # not ascending
    n = torch.tensor([20, 20], dtype=torch.int32, device=DEV)
    B.sirllm_compact_kv(cfg, dk, None, dk, None, keep.to(DEV), n, ws)
    assert B.sirllm_status(ws, clear=True) == B.STATUS_BAD_KEEP
    assert torch.equal(dk.cpu(), k)
    keep[1] = torch.arange(20) + 30                            # runs past the capacity
    B.sirllm_compact_kv(cfg, dk, None, dk, None, keep.to(DEV), n, ws)
    assert B.sirllm_status(ws, clear=True) == B.STATUS_BAD_KEEP
    assert torch.equal(dk.cpu(), k)


# ------------------------------------------------------------------------------- whole rounds

def _run_stream(w, rounds, ragged=False, seed=0, check_kv_host=True, rho=None, via_graph=False):
    st = DeviceState(w, seed=seed)
    graph = None
    twins = oracle_twin(w, st.decay.cpu())
    M = st.cfg.max_new
    for r in range(rounds):
        n_new = None
        if ragged:
            n_new = wl.ragged_lengths(seed, w.n_streams, r, w.new_tokens).tolist()
        n_new = st.fill_round(r, n_new, rho)
        # GPU scores first (the same kernel the fused round runs), for the oracle to rank
        e_gpu = torch.zeros_like(st.new_entropy)
        B.sirllm_score(st.cfg, st.logits, st.token_ids, st.n_new, e_gpu, st.ws)
        before = [t.live_len for t in twins]
        if via_graph and r > 0:
            if graph is None:   # the first round ran eagerly; every later one is a replay
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    st.enqueue_step()
                torch.cuda.current_stream().wait_stream(side)
            graph.replay()
            st.host_len = st.live_len.cpu().tolist()
        else:
            st.step()
        assert B.sirllm_status(st.ws) == 0
        e_gpu = e_gpu.cpu()
        for s, tw in enumerate(twins):
            T, l = n_new[s], before[s]
            rows = slice(s * M, s * M + T)
            want_e = oracle.score(st.logits[rows].cpu(), st.token_ids[rows].cpu())
            assert_entropy_close(e_gpu[rows], want_e)                          # P1
            assert torch.equal(st.new_entropy[rows].cpu().view(torch.int32),
                               e_gpu[rows].view(torch.int32))                  # fused == standalone
            serials = torch.arange(int(tw.next_serial.value), int(tw.next_serial.value) + T)
            tw.k[:, l:l + T] = wl.make_kv_rows(w, seed, "k", s, serials)
            tw.v[:, l:l + T] = wl.make_kv_rows(w, seed, "v", s, serials)
            keep = tw.step(e_gpu[rows])                                        # P2: same scores
            n = tw.live_len
            assert st.host_len[s] == n and int(st.n_keep[s]) == n
            assert torch.equal(st.keep_idx[s, :n].cpu(), keep)
            assert torch.equal(st.scores[s, :n].cpu().view(torch.int32), tw.E[:n].view(torch.int32))
            assert torch.equal(st.serial[s, :n].cpu(), tw.serial[:n])
            if check_kv_host:                                                  # P3
                assert torch.equal(st.k[s, :, :n].cpu(), tw.k[:, :n])
                assert torch.equal(st.v[s, :, :n].cpu(), tw.v[:, :n])
        st.check_kv_by_content()
    return st


def test_step_tiny_workload():
    st = _run_stream(wl.WORKLOADS["tiny"], 1)
    assert st.host_len == [256]


def test_step_multi_round_small_stream():
    w = wl.WORKLOADS["mistral_7b_gqa"].scaled(n_layers=2, n_kv_heads=3, capacity=1536, budget=1024,
                                              n_recent=128, new_tokens=200, vocab=5003)
    _run_stream(w, 12)


def test_step_ragged_multi_stream_rounds():
    w = wl.WORKLOADS["batched64"].scaled(n_streams=5, n_layers=2, n_kv_heads=2, capacity=512,
                                         budget=256, n_recent=64, new_tokens=100, vocab=4099)
    _run_stream(w, 10, ragged=True)


def test_step_paper_shaped_small_rounds():
    w = wl.WORKLOADS["rps_1024"].scaled(n_layers=2, n_kv_heads=2, vocab=32000)
    _run_stream(w, 30, rho=0.0)


@pytest.mark.parametrize("name,eta", [("dailydialog_512", 0.5), ("dailydialog_512", 0.6),
                                      ("dailydialog_512", 0.7), ("rps_1024", 0.7),
                                      ("rps_1024", 0.8), ("rps_1024", 0.9)])
def test_step_paper_cache_shapes_and_decay_ratios(name, eta):
    # the shapes and decay ratios of the paper's own runs: cache 512 = 4 sinks + 508 entropy slots,
    # ~120 tokens per round, decay 0.5 / 0.6 / 0.7 (Table 1); cache 1024 = 4 + 1020, 54 tokens per
    # round, decay 0.7 / 0.8 / 0.9 (Table 3); no recent window.  Whole rounds on fewer planes:
    # scores, keep lists, compacted scores, tags and K/V against the oracle every round.
    w = wl.WORKLOADS[name].scaled(n_layers=2, n_kv_heads=2, decay=eta)
    rounds = 24 if name == "dailydialog_512" else 40
    st = _run_stream(w, rounds)
    assert st.host_len == [w.budget]


def test_step_replayed_from_a_cuda_graph():
    # the round is three kernel launches chained by programmatic dependent launch and touches
    # no host state, so it can be captured once and replayed: every replayed round against the
    # oracle (ragged lengths arrive through device memory, not through the captured arguments)
    w = wl.WORKLOADS["batched64"].scaled(n_streams=3, n_layers=2, n_kv_heads=2, capacity=512,
                                         budget=256, n_recent=64, new_tokens=100, vocab=4099)
    _run_stream(w, 8, ragged=True, via_graph=True)
    w = wl.WORKLOADS["mistral_7b_gqa"].scaled(n_layers=8, n_kv_heads=8, capacity=1536, budget=1024,
                                              n_recent=128, new_tokens=200, vocab=5003)
    _run_stream(w, 8, via_graph=True)      # wide enough for the persistent gather


def _random_shape(seed: int):
    """A seeded random configuration: every size that a kernel tiles over is drawn, so that row
    widths, vocabulary tails, window splits and stream counts off the measured shapes are met."""
    import random
    g = random.Random(1000 + seed)
    head_dim = g.choice([8, 16, 40, 64, 80, 96, 128, 160, 256])
    n_streams = g.choice([1, 1, 2, 3, 5])
    wide = seed % 2 == 1          # enough planes and rows for the persistent (ring) gather
    budget = g.randrange(300, 700) if wide else g.randrange(8, 700)
    n_sink = g.randrange(0, min(9, budget + 1))
    n_recent = g.randrange(0, budget - n_sink + 1) if g.random() < 0.7 else 0
    if g.random() < 0.15:
        n_recent = budget - n_sink                       # k = 0: nothing chosen by score
    new_tokens = g.randrange(1, 2 * budget) if g.random() < 0.8 else g.randrange(1, 40)
    capacity = budget + new_tokens + g.randrange(0, 64)
    vocab = g.choice([g.randrange(2, 300), g.randrange(300, 9000), g.randrange(9000, 70000)])
    return wl.WORKLOADS["tiny"].scaled(
        name=f"random{seed}", n_streams=n_streams,
        n_layers=g.randrange(6, 13) if wide else g.randrange(1, 4),
        n_kv_heads=g.randrange(4, 9) if wide else g.randrange(1, 5), head_dim=head_dim, capacity=capacity, budget=budget,
        n_sink=n_sink, n_recent=n_recent, new_tokens=new_tokens, vocab=vocab,
        logits_dtype=g.choice(["f32", "bf16"]), kv_dtype=g.choice(["f16", "bf16"]),
        decay=g.choice([0.5, 0.7, 0.9, 1.0]), decay_hi=None)


@pytest.mark.parametrize("seed", range(16))
def test_step_random_configurations(seed):
    # whole rounds on drawn shapes (ragged lengths on the multi-stream ones): scores, keep lists,
    # compacted scores, tags and K/V against the oracle every round
    w = _random_shape(seed)
    rounds = max(4, min(12, 3 * w.budget // max(1, w.new_tokens) + 3))
    _run_stream(w, rounds, ragged=w.n_streams > 1, seed=seed)


def test_retained_tokens_overlap_with_a_run_on_the_oracles_own_scores():
    # Every other whole-round test hands the oracle the GPU's scores, so that index sets can be
    # compared bit for bit.  Here the oracle runs alone, on its OWN fp64-derived scores, and
    # the retained TOKENS (serial tags) are compared as sets: scores that differ in the last
    # fp32 digits may swap two near-equal candidates at the cut, nothing more.  The overlap
    # (intersection over union) is printed and must stay above 0.99 in every round.
    w = wl.WORKLOADS["mistral_7b_gqa"].scaled(n_layers=1, n_kv_heads=1, capacity=1536, budget=1024,
                                              n_recent=128, new_tokens=256, vocab=5003)
    st = DeviceState(w)
    tw = oracle_twin(w, st.decay.cpu(), with_kv=False)[0]
    worst = 1.0
    for r in range(16):
        st.fill_round(r)
        T = w.new_tokens
        st.step()
        assert B.sirllm_status(st.ws) == 0
        tw.step(oracle.score(st.logits[:T].cpu(), st.token_ids[:T].cpu()))
        n = tw.live_len
        assert st.host_len[0] == n
        got = set(st.serial[0, :n].cpu().tolist())
        want = set(tw.serial[:n].tolist())
        worst = min(worst, len(got & want) / len(got | want))
    print(f"retained-token overlap with the pure-oracle run, worst round: {worst:.5f}")
    assert worst > 0.99


def test_step_host_refused_call_leaves_the_device_untouched():
    # a bad value for the SECOND stream: nothing of the first stream may have been copied
    w = wl.WORKLOADS["batched64"].scaled(n_streams=2, n_layers=1, n_kv_heads=2, capacity=256,
                                         budget=128, n_recent=16, new_tokens=40, vocab=1000)
    st = DeviceState(w)
    st.fill_round(0)
    st.step()
    S, P, M, D = w.n_streams, w.planes_per_stream, w.new_tokens, w.head_dim
    h_logits = torch.full((S * M, w.vocab), 3.0, dtype=w.torch_logits_dtype).pin_memory()
    h_ids = torch.full((S * M,), 7, dtype=torch.int32).pin_memory()
    h_k = torch.full((S, P, M, D), 5.0, dtype=w.torch_kv_dtype).pin_memory()
    h_len = torch.tensor(st.host_len, dtype=torch.int32).pin_memory()
    h_keep = torch.zeros(S, st.cfg.threshold, dtype=torch.int32).pin_memory()
    h_nk = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_e = torch.zeros(S * M, dtype=torch.float32).pin_memory()
    snap = [t.clone() for t in (st.logits, st.token_ids, st.n_new, st.scores, st.serial, st.live_len,
                                st.k, st.v, st.keep_idx, st.n_keep, st.new_entropy)]
    for bad_new, bad_len in (([M, M + 1], None), ([M, -2], None), (None, [int(h_len[0]), -1])):
        h_n_new = torch.tensor(bad_new if bad_new else [M, M], dtype=torch.int32).pin_memory()
        lens = torch.tensor(bad_len, dtype=torch.int32).pin_memory() if bad_len else h_len
        with pytest.raises(B.SirllmError) as err:
            B.sirllm_step_host(st.cfg, h_logits, h_ids, h_n_new, h_k, h_k, lens, st.logits, st.token_ids,
                               st.n_new, st.scores, st.serial, st.live_len, st.decay, st.k, st.v,
                               st.keep_idx, st.n_keep, st.new_entropy, h_keep, h_nk, h_e, st.ws)
        assert err.value.code == B.ERR_BAD_CONFIG
    torch.cuda.synchronize()
    now = (st.logits, st.token_ids, st.n_new, st.scores, st.serial, st.live_len, st.k, st.v,
           st.keep_idx, st.n_keep, st.new_entropy)
    for before, after in zip(snap, now):
        assert torch.equal(before, after)
    assert B.sirllm_status(st.ws) == 0


def test_rounds_worked_by_hand_from_algorithm_1_on_the_device(golden_dir):
    # the seven hand-worked rounds of tests/golden/algorithm1_hand_trace.txt through
    # sirllm_decay_select + sirllm_compact_kv: expected values come from the file, not from the oracle
    from test_oracle_step import _read_trace
    head, rounds = _read_trace(f"{golden_dir}/algorithm1_hand_trace.txt")
    cap, D, P = 8, 8, 3
    cfg = B.make_config(1, P, 1, D, cap, int(head["budget"]), int(head["n_sink"]), int(head["n_recent"]),
                        4, 16, torch.float32, torch.float16, threshold=int(head["threshold"]))
    ws = B.new_workspace(cfg)
    scores = torch.zeros(1, cap, device=DEV)
    serial = torch.full((1, cap), -1, dtype=torch.int64, device=DEV)
    live = torch.zeros(1, dtype=torch.int32, device=DEV)
    decay = torch.tensor([head["decay"]], device=DEV)
    keep = torch.zeros(1, cfg.threshold, dtype=torch.int32, device=DEV)
    n_keep = torch.zeros(1, dtype=torch.int32, device=DEV)
    k = torch.zeros(1, P, cap, D, dtype=torch.float16, device=DEV)
    v = torch.zeros_like(k)
    nxt = 0
    for r in rounds:
        T, l = len(r["new"]), int(live[0])
        for t in range(T):
            scores[0, l + t] = r["new"][t]
            serial[0, l + t] = nxt
            k[0, :, l + t] = nxt
            v[0, :, l + t] = -nxt
            nxt += 1
        live[0] = l + T
        B.sirllm_decay_select(cfg, scores, serial, live, decay, keep, n_keep, True, ws)
        B.sirllm_compact_kv(cfg, k, v, k, v, keep, n_keep, ws)
        n = int(n_keep[0])
        assert int(live[0]) == n == len(r["kept"])
        assert keep[0, :n].tolist() == r["kept"]
        assert serial[0, :n].tolist() == r["tokens"]
        assert scores[0, :n].tolist() == r["scores"]
        for p in range(P):
            assert k[0, p, :n, 0].tolist() == [float(x) for x in r["tokens"]]
            assert v[0, p, :n, D - 1].tolist() == [-float(x) for x in r["tokens"]]
    assert B.sirllm_status(ws) == 0


def test_step_overflowing_round_is_skipped_and_flagged():
    w = wl.WORKLOADS["tiny"].scaled(n_streams=2, n_layers=1, n_kv_heads=1, capacity=300, budget=256,
                                    new_tokens=200, vocab=1000)
    st = DeviceState(w, threshold=300)            # no eviction below 300: the 2nd round cannot fit
    st.fill_round(0)
    st.step()
    assert st.host_len == [200, 200]
    snap = (st.scores.clone(), st.k.clone(), st.serial.clone())
    st.fill_round(1, [200, 50])
    st.step()
    assert B.sirllm_status(st.ws, clear=True) == B.STATUS_OVERFLOW
    assert st.host_len == [200, 250]
    assert torch.equal(st.scores[0], snap[0][0]) and torch.equal(st.k[0], snap[1][0])


# ------------------------------------------------------------------------------- scores from pairs

def _device_tile_pairs(logits, tile):
    """What a GEMM epilogue would emit: per-tile (max, sum exp(z - max)) in fp32 (torch ops,
    input preparation only)."""
    T, V = logits.shape
    n = (V + tile - 1) // tile
    z = torch.full((T, n * tile), float("-inf"), dtype=torch.float32, device=logits.device)
    z[:, :V] = logits.float()
    z = z.view(T, n, tile)
    m = z.max(dim=2).values
    s = torch.exp(z - m[:, :, None]).sum(dim=2)
    return torch.stack([m, s], dim=2).contiguous()


@pytest.mark.parametrize("tile", [128, 1000])
def test_score_pairs_matches_oracle_and_the_logits_path(tile):
    S, M, V = 2, 50, 32000
    cfg = _score_cfg(M, V, torch.bfloat16, n_streams=S)
    ws = B.new_workspace(cfg)
    g = torch.Generator().manual_seed(tile)
    logits = (torch.randn(S * M, V, generator=g) * 2.5).to(torch.bfloat16).to(DEV)
    ids = torch.randint(0, V, (S * M,), generator=g, dtype=torch.int32)
    ids[3], ids[60], ids[75] = -1, V, V          # row 75 lies beyond n_new[1]: never looked at
    d_ids = ids.to(DEV)
    n_new = torch.tensor([50, 17], dtype=torch.int32, device=DEV)
    pairs = _device_tile_pairs(logits, tile)
    target = logits.float()[torch.arange(S * M, device=DEV), d_ids.long().clamp(0, V - 1)].contiguous()
    out = torch.full((S * M,), -2.0, device=DEV)
    B.sirllm_score_pairs(cfg, pairs, target, d_ids, n_new, out, ws)
    assert B.sirllm_status(ws, clear=True) == B.STATUS_TOKEN_RANGE      # from row 60
    live = torch.zeros(S * M, dtype=torch.bool)
    live[:50] = True
    live[50:67] = True
    want = oracle.score_pairs(pairs.cpu(), target.cpu(), ids, V)
    assert_entropy_close(out.cpu()[live], want[live])
    assert (out.cpu()[~live] == -2.0).all() and float(out[3]) == 0.0 and float(out[60]) == 0.0
    ref = torch.zeros(S * M, device=DEV)
    B.sirllm_score(cfg, logits, d_ids, n_new, ref, ws)
    assert_entropy_close(out.cpu()[live], ref.cpu()[live])


def test_step_pairs_round_matches_oracle_and_the_logits_round():
    w = wl.WORKLOADS["mistral_7b_gqa"].scaled(n_layers=1, n_kv_heads=2, capacity=1024, budget=512,
                                              n_recent=64, new_tokens=300, vocab=8000)
    a, b = DeviceState(w), DeviceState(w)
    tw = oracle_twin(w, b.decay.cpu(), with_kv=False)[0]
    for r in range(4):
        a.fill_round(r)
        b.fill_round(r)
        a.step()
        pairs = _device_tile_pairs(b.logits, 256)
        target = b.logits.float()[torch.arange(b.logits.shape[0], device=DEV),
                                  b.token_ids.long()].contiguous()
        B.sirllm_step_pairs(b.cfg, pairs, target, b.token_ids, b.n_new, b.scores, b.serial, b.live_len,
                            b.decay, b.k, b.v, b.keep_idx, b.n_keep, b.new_entropy, b.ws)
        b.host_len = b.live_len.cpu().tolist()
        assert B.sirllm_status(b.ws) == 0
        e = b.new_entropy[:300].cpu()
        assert_entropy_close(e, oracle.score_pairs(pairs.cpu(), target.cpu(), b.token_ids.cpu(), w.vocab))
        assert_entropy_close(e, a.new_entropy[:300])            # the logits path agrees
        keep = tw.step(e)                                       # the oracle ranks the same scores
        n = tw.live_len
        assert b.host_len == [n] and a.host_len == [n]
        assert torch.equal(b.keep_idx[0, :n].cpu(), keep)
        assert torch.equal(b.scores[0, :n].cpu().view(torch.int32), tw.E[:n].view(torch.int32))
        assert torch.equal(b.serial[0, :n].cpu(), tw.serial[:n])
        b.check_kv_by_content()


# ------------------------------------------------------------------------------- sharded forms

@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_score_partial_over_uneven_column_ranges_matches_oracle(dtype):
    # a vocabulary-parallel LM head: every "rank" (here: one call each, on one device) reduces
    # its column range to a pair and a target logit per row; the pairs of all ranges then give
    # the scores.  Ranges are uneven, start off the 16-byte grid, one is empty, one is a few
    # columns wide and one needs several CTAs per row.
    S, M, V = 2, 30, 70001
    ranges = [(0, 5), (5, 40001), (40001, 40001), (40001, V)]
    cfg = _score_cfg(M, V, dtype, n_streams=S)
    ws = B.new_workspace(cfg)
    g = torch.Generator().manual_seed(3)
    logits = (torch.randn(S * M, V, generator=g) * 2.5).to(dtype)
    logits[4, 10:30000] = -float("inf")                   # masked stretch inside one range
    ids = torch.randint(0, V, (S * M,), generator=g, dtype=torch.int32)
    ids[1], ids[2], ids[5], ids[6] = -1, 3, 40000, 40001  # no prediction; range edges
    n_new = torch.tensor([M, 11], dtype=torch.int32)
    d_logits, d_ids, d_n = logits.to(DEV), ids.to(DEV), n_new.to(DEV)
    pairs = torch.full((S * M, len(ranges), 2), -9.0, device=DEV)
    targets = torch.full((len(ranges), S * M), -9.0, device=DEV)
    for r, (v0, v1) in enumerate(ranges):
        B.sirllm_score_partial(cfg, d_logits[:, v0:v1], v0, d_ids, d_n, pairs, targets[r], ws, pair_column=r)
    live = torch.zeros(S * M, dtype=torch.bool)
    live[:M] = True
    live[M:M + 11] = True
    assert (pairs.cpu()[~live] == -9.0).all() and (targets.cpu()[:, ~live] == -9.0).all()
    for r, (v0, v1) in enumerate(ranges):                 # each range against the oracle's pair
        want_p, want_t = oracle.range_pairs(logits, ids, v0, v1)
        got_p = pairs[:, r].cpu()
        assert torch.equal(targets[r].cpu()[live], want_t[live])
        empty = want_p[:, 1] == 0
        assert (got_p[empty & live] == 0).all()
        ok = live & ~empty
        if not ok.any():
            continue
        lse_got = got_p[ok, 0].double() + got_p[ok, 1].double().log()     # log of the range's sum
        lse_want = want_p[ok, 0].double() + want_p[ok, 1].double().log()
        assert float((lse_got - lse_want).abs().max()) < 2e-6
        assert float((got_p[ok, 0] - want_p[ok, 0]).abs().max()) < 1e-5   # m ~ the range's maximum
    target = targets.clone()
    target[:, ~live.to(DEV)] = 0
    target = target.sum(dim=0)
    out = torch.full((S * M,), -2.0, device=DEV)
    B.sirllm_score_pairs(cfg, pairs, target, d_ids, d_n, out, ws)
    assert B.sirllm_status(ws) == 0
    want = oracle.score(logits, ids)
    assert_entropy_close(out.cpu()[live], want[live])
    ref = torch.zeros(S * M, device=DEV)                  # and against the single-GPU kernel
    B.sirllm_score(cfg, d_logits, d_ids, d_n, ref, ws)
    assert_entropy_close(out.cpu()[live], ref.cpu()[live])


@pytest.mark.parametrize("by", ["layers", "heads"])
def test_plane_sharded_rounds_equal_the_full_configuration(by):
    # tensor- / pipeline-parallel layouts: every rank holds a replica of the scores and the K/V
    # planes of some layers or heads.  Two such ranks (run one after the other on one device),
    # each with its own workspace and its own half of the planes, must produce the keep lists,
    # scores and tags of the unsharded run and, between them, its K/V - all of it the oracle's.
    from paper_2405_12528_b200 import sharding
    w = wl.WORKLOADS["mistral_7b_gqa"].scaled(n_streams=2, n_layers=4, n_kv_heads=2, capacity=768,
                                              budget=512, n_recent=64, new_tokens=150, vocab=4001)
    full = DeviceState(w)
    twins = oracle_twin(w, full.decay.cpu(), with_kv=False)
    world = 2
    ranks = []
    for r in range(world):
        layers, heads = sharding.plane_shard(w.n_layers, w.n_kv_heads, world, r, by)
        st = DeviceState(w.scaled(n_layers=len(layers), n_kv_heads=len(heads)))
        planes = torch.tensor([l * w.n_kv_heads + h for l in layers for h in heads], device=DEV)
        ranks.append((st, planes))
    for rnd in range(8):
        n_new = full.fill_round(rnd, wl.ragged_lengths(5, w.n_streams, rnd, w.new_tokens).tolist())
        for st, planes in ranks:                          # the same round on every rank
            st.logits.copy_(full.logits)
            st.token_ids.copy_(full.token_ids)
            st.n_new.copy_(full.n_new)
            for s in range(w.n_streams):
                l, T = st.host_len[s], n_new[s]
                st.serial[s, l:l + T] = full.serial[s, l:l + T]
                st.k[s, :, l:l + T] = full.k[s, planes, l:l + T]
                st.v[s, :, l:l + T] = full.v[s, planes, l:l + T]
        full.step()
        for st, _ in ranks:
            st.step()
            assert B.sirllm_status(st.ws) == 0 and st.host_len == full.host_len
        e = full.new_entropy.cpu()
        M = full.cfg.max_new
        for s, tw in enumerate(twins):
            n = full.host_len[s]
            for st, planes in ranks:
                assert torch.equal(st.keep_idx[s, :n], full.keep_idx[s, :n])
                assert torch.equal(st.scores[s, :n].view(torch.int32), full.scores[s, :n].view(torch.int32))
                assert torch.equal(st.serial[s, :n], full.serial[s, :n])
                assert torch.equal(st.k[s, :, :n], full.k[s, planes, :n])
                assert torch.equal(st.v[s, :, :n], full.v[s, planes, :n])
            keep = tw.step(e[s * M:s * M + n_new[s]])     # the oracle ranks the same scores
            assert tw.live_len == n and torch.equal(full.keep_idx[s, :n].cpu(), keep)
            assert torch.equal(full.scores[s, :n].cpu().view(torch.int32), tw.E[:n].view(torch.int32))
        full.check_kv_by_content()                        # K/V rows follow their tokens


# ------------------------------------------------------------------------------- comparison policies

@pytest.mark.parametrize("policy", [B.POLICY_STREAM, B.POLICY_RANDOM, B.POLICY_INTERVAL])
def test_keep_policy_matches_oracle_and_feeds_the_gather(policy):
    # StreamLLM / RandomLLM / IntervalLLM of Section 4.1.1: keep lists bit exact, then the same
    # K/V gather; streams with different lengths, one under the threshold
    lens = [1078, 1025, 3000, 640, 0]
    S, cap, budget, n_sink, n_recent = len(lens), 3072, 1024, 4, 0
    for n_recent in (0, 37):
        cfg = B.make_config(S, 2, 1, 64, cap, budget, n_sink, n_recent, 0, 16, torch.float32, torch.bfloat16)
        ws = B.new_workspace(cfg)
        live = torch.tensor(lens, dtype=torch.int32, device=DEV)
        keep = torch.full((S, budget), -1, dtype=torch.int32, device=DEV)
        nk = torch.zeros(S, dtype=torch.int32, device=DEV)
        g = torch.Generator().manual_seed(policy)
        k = torch.randn(S, 2, cap, 64, generator=g).to(torch.bfloat16)
        dk = k.to(DEV)
        B.sirllm_keep_policy(cfg, policy, live, 1234567890123, 5, 10, keep, nk, ws)
        B.sirllm_compact_kv(cfg, dk, None, dk, None, keep, nk, ws)
        assert B.sirllm_status(ws) == 0
        assert live.cpu().tolist() == lens
        for s, l in enumerate(lens):
            want = oracle.keep_policy(policy, l, n_sink, n_recent, budget, seed=1234567890123,
                                      stream=10 + s, rnd=5)
            n = int(nk[s])
            assert n == len(want)
            assert torch.equal(keep[s, :n].cpu(), want)
            for p in range(2):
                assert torch.equal(dk[s, p, :n].cpu(), oracle.gather_rows(k[s, p], want))


def test_step_long_stream_without_reset_keeps_denormal_scores():
    # The Rock-Paper-Scissors runs keep one cache for 2000 rounds of ~54 tokens (Table 7,
    # Section 4.2.3) with 4 sinks + 1020 entropy slots and no recent window; here 2000 rounds at
    # decay 0.7 on fewer planes.  The sink tokens are never evicted, so their scores decay through
    # the denormal range and stick at the smallest denormal (0.7 * 2^-149 rounds back to 2^-149):
    # flushing denormals to zero on the device would break bit parity here.
    w = wl.WORKLOADS["rps_1024"].scaled(n_layers=1, n_kv_heads=2, vocab=2003, decay=0.7,
                                        budget=260, capacity=320)
    st = DeviceState(w)
    tw = oracle_twin(w, st.decay.cpu(), with_kv=False)[0]
    for r in range(2000):
        st.fill_round(r)
        st.step()
        e = st.new_entropy[:w.new_tokens].cpu()
        keep = tw.step(e)
        n = tw.live_len
        assert st.host_len == [n]
        assert torch.equal(st.keep_idx[0, :n].cpu(), keep), r
        assert torch.equal(st.scores[0, :n].cpu().view(torch.int32), tw.E[:n].view(torch.int32)), r
        assert torch.equal(st.serial[0, :n].cpu(), tw.serial[:n]), r
        if r % 200 == 199:
            st.check_kv_by_content()
            assert_entropy_close(e, oracle.score(st.logits[:w.new_tokens].cpu(), st.token_ids[:w.new_tokens].cpu()))
    assert B.sirllm_status(st.ws) == 0
    st.check_kv_by_content()
    assert st.scores[0, :4].cpu().view(torch.int32).tolist() == [1, 1, 1, 1]     # 2^-149
    # with decay < 1 nothing old survives (Appendix B): the cache holds only recent serials
    newest = int(st.serial[0, :n].max())
    assert int(st.serial[0, 4]) > newest - 40 * w.new_tokens


def test_select_randomised_shapes_and_score_patterns():
    # many seeded draws of (lengths, sinks, recent, budget, threshold, decay) and of score
    # patterns that steer the selection kernel through all its branches: narrow key ranges (one
    # short digit), bulk ties (several digit passes), few distinct values, negative and zero
    # scores, k = 1 and k = all-but-one
    rng = np.random.default_rng(12345)
    for case in range(60):
        cap = int(rng.choice([64, 300, 1000, 4096, 9000]))
        n_sink = int(rng.integers(0, 6))
        n_recent = int(rng.integers(0, max(1, cap // 8)))
        k = int(rng.choice([0, 1, 2, int(rng.integers(1, max(2, cap // 2)))]))
        budget = max(1, n_sink + n_recent + k)
        if budget > cap:
            continue
        threshold = int(min(cap, budget + rng.choice([0, 0, 3, cap // 10])))
        S = int(rng.integers(1, 5))
        lens = [int(rng.integers(0, cap + 1)) for _ in range(S)]
        lens[0] = int(min(cap, budget + 1 + rng.integers(0, max(1, cap - budget))))   # evicts
        if rng.random() < 0.3:
            lens[-1] = min(cap, threshold + 1)                                          # evicts one
        cfg = B.make_config(S, 1, 1, 8, cap, budget, n_sink, n_recent, 0, 16, torch.float32,
                            torch.bfloat16, threshold=threshold)
        ws = B.new_workspace(cfg)
        E = torch.zeros(S, cap)
        pattern = case % 6
        for s, l in enumerate(lens):
            u = torch.tensor(rng.random(l), dtype=torch.float32)
            if pattern == 0:
                E[s, :l] = u * 12
            elif pattern == 1:
                E[s, :l] = 3.0 + u * 1e-5                      # narrow range
            elif pattern == 2:
                E[s, :l] = torch.round(u * 3)                  # 4 distinct values: bulk ties
            elif pattern == 3:
                E[s, :l] = (u - 0.5) * 4                       # negatives too
            elif pattern == 4:
                E[s, :l] = torch.where(u < 0.7, torch.zeros(()), u)   # mostly exact zeros
            else:
                E[s, :l] = torch.exp((u - 0.5) * 60)           # 26 orders of magnitude
        decay = [float(rng.choice([1.0, 0.9, 0.5])) for _ in range(S)]
        serial = torch.arange(S * cap, dtype=torch.int64).view(S, cap)
        dE, dser = E.to(DEV), serial.to(DEV)
        dlen = torch.tensor(lens, dtype=torch.int32, device=DEV)
        keep = torch.full((S, threshold), -1, dtype=torch.int32, device=DEV)
        nk = torch.zeros(S, dtype=torch.int32, device=DEV)
        B.sirllm_decay_select(cfg, dE, dser, dlen, torch.tensor(decay, device=DEV), keep, nk, 1, ws)
        assert B.sirllm_status(ws) == 0
        for s, l in enumerate(lens):
            Es = E[s].clone()
            oracle.decay(Es, l, decay[s])
            want = oracle.select(Es, l, n_sink, n_recent, budget, threshold)
            n = int(nk[s])
            ctx = (case, s, l, n_sink, n_recent, budget, threshold, pattern)
            assert n == len(want) == int(dlen[s]), ctx
            assert torch.equal(keep[s, :n].cpu(), want), ctx
            assert torch.equal(dE[s, :n].cpu().view(torch.int32), Es[want.long()].view(torch.int32)), ctx
            assert torch.equal(dser[s, :n].cpu(), serial[s][want.long()]), ctx


def test_step_with_optional_arguments_left_out():
    # no tags, no keep-list / count outputs (the workspace holds them), no raw-score output,
    # only K (V skipped), n_new = NULL meaning max_new everywhere
    w = wl.WORKLOADS["tiny"].scaled(n_streams=2, n_layers=1, n_kv_heads=2, capacity=256, budget=96,
                                    n_recent=16, new_tokens=70, vocab=3001)
    a, b = DeviceState(w), DeviceState(w)
    for r in range(3):
        a.fill_round(r)
        b.fill_round(r)
        a.step()
        B.sirllm_step(b.cfg, b.logits, b.token_ids, None, b.scores, None, b.live_len, b.decay,
                      b.k, None, None, None, None, b.ws)
        assert B.sirllm_status(b.ws) == 0
        assert torch.equal(a.live_len, b.live_len)
        n = int(a.live_len[0])
        assert torch.equal(a.scores[:, :n].view(torch.int32), b.scores[:, :n].view(torch.int32))
        assert torch.equal(a.k[:, :, :n], b.k[:, :, :n])
        b.host_len = b.live_len.cpu().tolist()
    # V was never compacted on b: its new rows still sit where they were appended
    assert not torch.equal(a.v[:, :, :n], b.v[:, :, :n])


def test_step_host_matches_the_device_round():
    # the same rounds once with device-resident inputs and once through sirllm_step_host
    # (pinned host logits / ids / new K/V rows in, keep lists / lengths / raw scores out)
    w = wl.WORKLOADS["batched64"].scaled(n_streams=3, n_layers=2, n_kv_heads=2, capacity=384,
                                         budget=192, n_recent=32, new_tokens=80, vocab=2500)
    a, b = DeviceState(w), DeviceState(w)
    S, P, M, D = w.n_streams, w.planes_per_stream, w.new_tokens, w.head_dim
    h_len = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_keep = torch.zeros(S, b.cfg.threshold, dtype=torch.int32).pin_memory()
    h_nk = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_e = torch.zeros(S * M, dtype=torch.float32).pin_memory()
    next_serial = 0
    for r in range(5):
        n_new = wl.ragged_lengths(3, S, r, M).tolist()
        a.fill_round(r, n_new)
        a.step()
        # host copies of the round's inputs, generated on the CPU
        h_logits = torch.zeros(S * M, w.vocab, dtype=w.torch_logits_dtype).pin_memory()
        h_ids = torch.zeros(S * M, dtype=torch.int32).pin_memory()
        h_k = torch.zeros(S, P, M, D, dtype=w.torch_kv_dtype).pin_memory()
        h_v = torch.zeros(S, P, M, D, dtype=w.torch_kv_dtype).pin_memory()
        for s in range(S):
            T = n_new[s]
            h_logits[s * M:s * M + T] = wl.make_logits(w, 0, s, r, T)
            h_ids[s * M:s * M + T] = wl.make_token_ids(w, 0, s, r, T)
            serials = torch.arange(b.next_serial[s], b.next_serial[s] + T)
            h_k[s, :, :T] = wl.make_kv_rows(w, 0, "k", s, serials)
            h_v[s, :, :T] = wl.make_kv_rows(w, 0, "v", s, serials)
            l = int(h_len[s])
            b.serial[s, l:l + T] = serials.to(DEV)          # tags are device state of the caller
            b.next_serial[s] += T
        h_n_new = torch.tensor(n_new, dtype=torch.int32).pin_memory()
        B.sirllm_step_host(b.cfg, h_logits, h_ids, h_n_new, h_k, h_v, h_len, b.logits, b.token_ids,
                           b.n_new, b.scores, b.serial, b.live_len, b.decay, b.k, b.v, b.keep_idx,
                           b.n_keep, b.new_entropy, h_keep, h_nk, h_e, b.ws)
        torch.cuda.current_stream().synchronize()
        assert B.sirllm_status(b.ws) == 0
        assert h_nk.tolist() == a.host_len == b.live_len.cpu().tolist()
        h_len.copy_(h_nk)
        for s in range(S):
            n, T = a.host_len[s], n_new[s]
            assert torch.equal(h_keep[s, :n], a.keep_idx[s, :n].cpu())
            assert torch.equal(h_e[s * M:s * M + T].view(torch.int32),
                               a.new_entropy[s * M:s * M + T].cpu().view(torch.int32))
            assert torch.equal(a.scores[s, :n].view(torch.int32), b.scores[s, :n].view(torch.int32))
            assert torch.equal(a.serial[s, :n], b.serial[s, :n])
            assert torch.equal(a.k[s, :, :n], b.k[s, :, :n]) and torch.equal(a.v[s, :, :n], b.v[s, :, :n])


# ------------------------------------------------------------------------------- rotary re-indexing

def _ordered16(t):
    b = t.view(torch.int16).to(torch.int32)
    return torch.where(b < 0, -(b & 0x7FFF), b)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("layout", [B.ROPE_HALF, B.ROPE_INTERLEAVED])
def test_rerotate_keys_matches_oracle(dtype, layout):
    # both sides rotate in fp64 and round once, from fp64, to the 16-bit type: results agree bit
    # for bit except where the last bits of the fp64 value (the device's sincos and fused product) put a
    # value on the other side of a rounding boundary - one unit in the last place, rarely
    S, P, cap, D, thr = 2, 3, 700, 128, 400
    cfg = B.make_config(S, P, 1, D, cap, thr, 0, 0, 0, 16, torch.float32, dtype)
    g = torch.Generator().manual_seed(layout + 7)
    k = (torch.randn(S, P, cap, D, generator=g) * 2).to(dtype)
    n_list = [400, 123]
    keep = torch.full((S, thr), -1, dtype=torch.int32)
    for s, n in enumerate(n_list):
        picked = torch.sort(torch.randperm(cap - 20, generator=g)[:n - 20]).values + 20
        keep[s, :n] = torch.cat([torch.arange(20), picked]).to(torch.int32)    # 20 rows stay put
    dk = k.to(DEV)
    B.sirllm_rerotate_keys(cfg, dk, keep.to(DEV), torch.tensor(n_list, dtype=torch.int32, device=DEV),
                           10000.0, layout)
    got = dk.cpu()
    n_elems = n_off = 0
    for s, n in enumerate(n_list):
        for p in range(P):
            want = oracle.rerotate_plane(k[s, p], keep[s, :n], 10000.0, layout)
            assert torch.equal(got[s, p, n:], k[s, p, n:])                     # beyond the live rows
            assert torch.equal(got[s, p, :20], k[s, p, :20])                   # rows that did not move
            d = (_ordered16(got[s, p, :n]) - _ordered16(want[:n])).abs()
            assert int(d.max()) <= 1
            n_off += int((d != 0).sum())
            n_elems += d.numel()
            assert not torch.equal(got[s, p, 20:n], k[s, p, 20:n])
    assert n_off <= 1e-3 * n_elems, (n_off, n_elems)


def _rerotate_case(S, P, cap, D, thr, n_list, fixed, dtype, layout, seed, scale=2.0, exponent_spread=0,
                   base=10000.0):
    """Random keys, keep lists whose first `fixed` rows stay put; every plane against the oracle."""
    cfg = B.make_config(S, P, 1, D, cap, thr, 0, 0, 0, 16, torch.float32, dtype)
    g = torch.Generator().manual_seed(seed)
    k = torch.randn(S, P, cap, D, generator=g) * scale
    if exponent_spread:                  # magnitudes spread over many binades, down into the subnormals
        k = k * torch.exp2(-torch.randint(0, exponent_spread, k.shape, generator=g).float())
    k = k.to(dtype)
    keep = torch.full((S, thr), -1, dtype=torch.int32)
    for s, n in enumerate(n_list):
        f = min(fixed, n)
        picked = torch.sort(torch.randperm(cap - f, generator=g)[:n - f]).values + f
        keep[s, :n] = torch.cat([torch.arange(f), picked]).to(torch.int32)
    dk = k.to(DEV)
    B.sirllm_rerotate_keys(cfg, dk, keep.to(DEV), torch.tensor(n_list, dtype=torch.int32, device=DEV),
                           base, layout)
    got = dk.cpu()
    n_elems = n_off = 0
    for s, n in enumerate(n_list):
        for p in range(P):
            want = oracle.rerotate_plane(k[s, p], keep[s, :n], base, layout)
            assert torch.equal(got[s, p, n:], k[s, p, n:])                     # beyond the live rows
            d = (_ordered16(got[s, p, :n]) - _ordered16(want[:n])).abs()
            assert int(d.max()) <= 1 if n else True
            n_off += int((d != 0).sum())
            n_elems += d.numel()
    assert n_off <= 1e-3 * max(n_elems, 1), (n_off, n_elems)
    return n_off, n_elems


@pytest.mark.parametrize("layout", [B.ROPE_HALF, B.ROPE_INTERLEAVED])
def test_rerotate_work_split_over_streams_row_groups_and_planes(layout):
    # the kernel cuts (stream, row group, plane) lists into equal shares per block: many short
    # streams, streams that moved nothing or are empty, one long stream with few planes, plane
    # counts that no share divides, row widths with 5, 16 and 32 threads per row
    _rerotate_case(9, 5, 90, 64, 64, [64, 0, 17, 64, 1, 33, 64, 2, 50], 3, torch.bfloat16, layout, 31)
    _rerotate_case(3, 7, 300, 80, 200, [200, 199, 200], 200, torch.float16, layout, 32)   # nothing moved
    _rerotate_case(1, 1, 9000, 128, 6000, [6000], 2500, torch.bfloat16, layout, 33)
    _rerotate_case(2, 13, 400, 256, 256, [256, 101], 0, torch.float16, layout, 34)
    _rerotate_case(1, 3, 200, 512, 128, [77], 5, torch.bfloat16, layout, 35)
    _rerotate_case(40, 2, 64, 16, 48, [48 - (s % 5) for s in range(40)], 1, torch.bfloat16, layout, 36)
    # shifts of tens of thousands of positions (the largest cache the library takes) at a large base
    _rerotate_case(1, 2, 49152, 128, 600, [600], 0, torch.bfloat16, layout, 37, base=500000.0)
    _rerotate_case(1, 1, 49152, 64, 300, [300], 0, torch.float16, layout, 38, base=1.0e6)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_rerotate_rounds_tiny_and_subnormal_results_once(dtype):
    # keys spread over 60 binades, ending below the smallest normal number of the type (and, for
    # bf16, of fp32): results that are subnormal, that cancel to almost nothing or round to zero
    # must still be the fp64 rotation rounded once
    scale = 2.0 ** -100 if dtype == torch.bfloat16 else 2.0 ** -4
    exact_zero = _rerotate_case(2, 3, 500, 128, 300, [300, 210], 4, dtype, B.ROPE_HALF, 41, scale, 40)
    assert exact_zero[1] > 0
    _rerotate_case(1, 2, 260, 64, 200, [200], 0, dtype, B.ROPE_INTERLEAVED, 42, scale, 40)
    # rows of zeros (padding) stay zeros
    cfg = B.make_config(1, 2, 1, 64, 100, 50, 0, 0, 0, 16, torch.float32, dtype)
    z = torch.zeros(1, 2, 100, 64, dtype=dtype, device=DEV)
    keep = (torch.arange(50, dtype=torch.int32) * 2).view(1, 50).to(DEV)
    B.sirllm_rerotate_keys(cfg, z, keep, torch.tensor([50], dtype=torch.int32, device=DEV), 10000.0, B.ROPE_HALF)
    assert int(z.view(torch.int16).abs().max()) == 0


def test_rerotate_after_compaction_equals_keys_written_at_their_new_positions():
    # keys are stored rotated for the slot they were written to; after eviction + re-indexing
    # every kept key must equal (to storage rounding) the same token's key rotated for its new slot
    S, P, cap, D, n = 1, 2, 300, 64, 180
    cfg = B.make_config(S, P, 1, D, cap, n, 0, 0, 0, 16, torch.float32, torch.float16)
    ws = B.new_workspace(cfg)
    g = torch.Generator().manual_seed(11)
    raw = torch.randn(P, cap, D, generator=g, dtype=torch.float64)              # keys before rotation
    stored = torch.stack([torch.stack([oracle.rope_rotate(raw[p, j], j, 10000.0, B.ROPE_HALF)
                                       for j in range(cap)]) for p in range(P)]).to(torch.float16)
    keep = torch.sort(torch.randperm(cap, generator=g)[:n]).values.to(torch.int32).view(1, n)
    dk = stored.view(1, P, cap, D).to(DEV)
    nk = torch.tensor([n], dtype=torch.int32, device=DEV)
    B.sirllm_compact_kv(cfg, dk, None, dk, None, keep.to(DEV), nk, ws)
    B.sirllm_rerotate_keys(cfg, dk, keep.to(DEV), nk, 10000.0, B.ROPE_HALF)
    got = dk.cpu()[0].double()
    for p in range(P):
        for j in range(0, n, 7):
            fresh = oracle.rope_rotate(raw[p, int(keep[0, j])], j, 10000.0, B.ROPE_HALF)
            assert torch.allclose(got[p, j], fresh, rtol=0, atol=8e-3)          # two fp16 roundings


def test_compact_in_place_with_planes_cut_into_many_chained_segments():
    # few planes and long keep lists: every plane is cut into the maximum number of segments
    # that different SMs take, so correctness rests on the progress-word chain; large and small
    # displacements, a stream that moves nothing and one that moves a single row
    _compact_case(4, 1, 20000, 128, [15000, 19999, 20000, 2], True, 21)
    _compact_case(1, 2, 49152, 64, [30000], True, 22)
    # out of place with the same cut (no chain needed, all rows copied)
    _compact_case(2, 1, 20000, 128, [15000, 777], False, 23)


def test_a_device_side_wait_that_runs_out_is_reported_not_hung():
    # failure detection without a failure: the library's bounded wait polls a progress word that
    # nothing sets, gives up, raises the status bit, and the context keeps working
    w = wl.WORKLOADS["tiny"].scaled(n_layers=1, n_kv_heads=1, capacity=128, budget=64, n_recent=8,
                                    new_tokens=40, vocab=501)
    st = DeviceState(w)
    B.sirllm_selftest_bounded_wait(st.cfg, st.ws, 2000)
    assert B.sirllm_status(st.ws, clear=True) == B.STATUS_TIMEOUT
    assert B.sirllm_status(st.ws) == 0
    for r in range(3):                      # the same workspace still runs rounds correctly
        st.fill_round(r)
        st.step()
    assert B.sirllm_status(st.ws) == 0
    st.check_kv_by_content()
    assert st.host_len == [64]


def test_prepared_call_repeats_the_checked_call():
    # arguments are checked and marshalled once; every later invocation issues the same call on
    # whatever the tensors hold by then
    w = wl.WORKLOADS["tiny"].scaled(n_layers=1, n_kv_heads=2, capacity=256, budget=96, n_recent=16,
                                    new_tokens=70, vocab=3001)
    a, b = DeviceState(w), DeviceState(w)
    step = B.prepared(B.sirllm_step, b.cfg, b.logits, b.token_ids, b.n_new, b.scores, b.serial, b.live_len,
                      b.decay, b.k, b.v, b.keep_idx, b.n_keep, b.new_entropy, b.ws)
    for r in range(4):
        a.fill_round(r)
        b.fill_round(r)
        a.step()
        step()
        b.host_len = b.live_len.cpu().tolist()
        assert a.host_len == b.host_len
        n = a.host_len[0]
        assert torch.equal(a.keep_idx[:, :n], b.keep_idx[:, :n])
        assert torch.equal(a.scores[:, :n].view(torch.int32), b.scores[:, :n].view(torch.int32))
        assert torch.equal(a.k[:, :, :n], b.k[:, :, :n]) and torch.equal(a.v[:, :, :n], b.v[:, :, :n])
    with pytest.raises(B.SirllmError):                       # the checks still run, once
        B.prepared(B.sirllm_step, b.cfg, b.logits, b.token_ids[:5], b.n_new, b.scores, b.serial, b.live_len,
                   b.decay, b.k, b.v, b.keep_idx, b.n_keep, b.new_entropy, b.ws)
