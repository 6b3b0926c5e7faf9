#!/usr/bin/env python
"""Throughput of the SirLLM retention pass (score -> append -> decay -> select -> compact).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one evicting round of the whole pass over one batch of synthetic input at steady
state (live length = budget before the round's tokens arrive).  One JSON line is printed by
rank 0.  With N > 1 every rank drives its own GPU with its own independent streams (the
pass shards by stream; there is no collective on the data path) and the line reports the
whole job: weak scaling.  The N ranks come from torchrun (RANK / WORLD_SIZE in the
environment) or, when the script is started plainly with --gpus N, from N child processes
it starts itself, one per GPU.

Timing: CUDA events on the launching stream, barrier + synchronize on both sides, max over
ranks.  The K timed rounds run back to back; every round reads a logits tensor (>= 1 GB on
the default workload) and a K/V cache (>= 2 GB) far larger than the 126 MB L2, and
rotates through as many logits tensors as it takes to hold twice the L2 (two on the default
workload, dozens on the workloads with short rounds), so nothing it needs is cache resident.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_12528_b200 import sharding  # noqa: E402
from paper_2405_12528_b200 import workloads as wl  # noqa: E402

METRIC = "tokens/s through entropy+decay+top-k eviction; KV compaction GB/s vs HBM peak"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "llama3_8b"      # the shape the 70 %-of-HBM target is quoted on
FALLBACK_HBM_GBS = 6650.0


# DRAM traffic of the dominant kernel from one ncu capture (profiles/compact_kernel_mistral_7b_gqa.md):
# dram__bytes_read.sum + dram__bytes_write.sum of ONE gather launch on mistral_7b_gqa (1.07 GB
# moved, 2.1 GB of cache on the device: only ~5 % of the written rows are still in L2 when the
# kernel ends, so the figure is close to what a full-size launch sends to DRAM).  Traffic grows
# in proportion to the moved bytes, so it is scaled to the timed launch; it is reported only
# while the kernel's source file is the one the counters were taken on.
NCU_CAPTURE = {"kernel": "compact_kernel", "workload": "mistral_7b_gqa",
               "dram_bytes": 536590592 + 483479808, "algorithmic_bytes": 2 * 4092 * 256 * 512,
               "sources": {"paper_2405_12528_b200/csrc/compact.cu": "5d3d22e8a1dc3b3c1bbd622d7cdec1b133a12df8"}}


def ncu_traffic(bytes_per_launch):
    import hashlib
    for rel, want in NCU_CAPTURE["sources"].items():
        try:
            with open(os.path.join(ROOT, rel), "rb") as fh:
                b = fh.read()
        except OSError:
            return None
        if hashlib.sha1(b"blob %d\0" % len(b) + b).hexdigest() != want:
            return None          # the kernel changed since the counters were taken
    return round(NCU_CAPTURE["dram_bytes"] * bytes_per_launch / NCU_CAPTURE["algorithmic_bytes"])


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "10"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        self.result = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            self.result = {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm),
                           "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------

class Pass:
    """Device state of one rank and the calls of one round."""

    def __init__(self, w: wl.Workload, seed: int, dev: str, stream_ids=None):
        from paper_2405_12528_b200 import binding as B
        self.B, self.w, self.seed, self.dev = B, w, seed, dev
        # global ids of the streams this rank hosts: they key the seeded inputs
        self.sid = list(stream_ids) if stream_ids is not None else list(range(w.n_streams))
        self.cfg = B.config_from_workload(w)
        S, P, C, D, M = w.n_streams, w.planes_per_stream, w.capacity, w.head_dim, w.new_tokens
        self.ws = B.new_workspace(self.cfg, dev)
        self.scores = torch.zeros(S, C, dtype=torch.float32, device=dev)
        self.serial = torch.full((S, C), -1, dtype=torch.int64, device=dev)
        self.live_len = torch.zeros(S, dtype=torch.int32, device=dev)
        self.decay = wl.stream_decay(w.scaled(n_streams=max(self.sid) + 1), seed)[self.sid].to(dev)
        self.keep_idx = torch.zeros(S, self.cfg.threshold, dtype=torch.int32, device=dev)
        self.n_keep = torch.zeros(S, dtype=torch.int32, device=dev)
        self.new_entropy = torch.zeros(S * M, dtype=torch.float32, device=dev)
        self.k = torch.zeros(S, P, C, D, dtype=w.torch_kv_dtype, device=dev)
        self.v = torch.zeros(S, P, C, D, dtype=w.torch_kv_dtype, device=dev)
        self.n_new = torch.full((S,), M, dtype=torch.int32, device=dev)
        bias = wl.zipf_bias_table(w.vocab, w.zipf_bias, dev) if w.zipf_bias else None
        self.pool = []                    # rounds of logits / ids to rotate through
        for r in range(logits_pool_size(w)):
            lg = torch.empty(S * M, w.vocab, dtype=w.torch_logits_dtype, device=dev)
            ids = torch.empty(S * M, dtype=torch.int32, device=dev)
            for s in range(S):
                wl.make_logits(w, seed, self.sid[s], r, M, dev, bias, out=lg[s * M:(s + 1) * M])
                ids[s * M:(s + 1) * M] = wl.make_token_ids(w, seed, self.sid[s], r, M, dev)
            self.pool.append((lg, ids))
        self.next_serial = 0
        self.round = 0
        # the fused round on either logits tensor, arguments checked and marshalled once
        self.fused = [B.prepared(B.sirllm_step, self.cfg, lg, ids, self.n_new, self.scores, self.serial,
                                 self.live_len, self.decay, self.k, self.v, self.keep_idx, self.n_keep,
                                 self.new_entropy, self.ws) for lg, ids in self.pool]

    def append_rows(self):
        """Stand-in for the model: writes the round's new K/V rows and tags behind the live rows."""
        w = self.w
        lens = self.live_len.cpu().tolist()
        T = w.new_tokens
        serials = torch.arange(self.next_serial, self.next_serial + T, device=self.dev)
        for s in range(w.n_streams):
            l = lens[s]
            self.serial[s, l:l + T] = serials
            self.k[s, :, l:l + T] = wl.make_kv_rows(w, self.seed, "k", self.sid[s], serials, device=self.dev)
            self.v[s, :, l:l + T] = wl.make_kv_rows(w, self.seed, "v", self.sid[s], serials, device=self.dev)
        self.next_serial += T

    def step(self, events=None):
        which = self.round % len(self.pool)
        self.round += 1
        if events is None:
            self.fused[which]()
        else:
            lg, ids = self.pool[which]
            self.B.sirllm_step_phases(self.cfg, lg, ids, self.n_new, self.scores, self.serial,
                                      self.live_len, self.decay, self.k, self.v, self.keep_idx,
                                      self.n_keep, self.new_entropy, self.ws, events)

    def prime(self):
        """Real rounds from an empty cache until the first eviction has happened."""
        w = self.w
        n = (w.budget + w.new_tokens - 1) // w.new_tokens + 1
        for _ in range(n):
            self.append_rows()
            self.step()
        assert self.live_len.cpu().tolist() == [w.budget] * w.n_streams
        assert self.B.sirllm_status(self.ws) == 0

    def moved_rows(self):
        """Rows that changed slot in the last round, summed over streams (in-place traffic)."""
        j = torch.arange(self.cfg.threshold, device=self.dev, dtype=torch.int32)
        moved = (self.keep_idx != j[None, :]) & (j[None, :] < self.n_keep[:, None])
        return int(moved.sum())


def step_bytes(w: wl.Workload, moved_rows: int) -> dict:
    """Algorithmic bytes of one round: logits read once (+ ids, target logit sector, score
    written), scores read+written, keep list; every moved K/V row read once and written once."""
    es = 4 if w.logits_dtype == "f32" else 2
    T = w.n_streams * w.new_tokens
    l = w.n_streams * (w.budget + w.new_tokens)
    score = T * w.vocab * es + T * (4 + 32 + 4)
    select = 2 * l * 4 + w.n_streams * w.budget * 4
    compact = 2 * moved_rows * w.row_bytes * 2 * w.planes_per_stream
    return {"score": score, "select": select, "compact": compact, "step": score + select + compact}


L2_BYTES = 126 << 20


def logits_pool_size(w: wl.Workload) -> int:
    """Logits tensors the timed rounds rotate through: at least two, and as many as it takes
    for the pool to hold twice the L2, so that no round finds its logits cache resident."""
    es = 4 if w.logits_dtype == "f32" else 2
    per_round = w.n_streams * w.new_tokens * w.vocab * es
    return max(2, min(96, -(-2 * L2_BYTES // per_round)))


def config_dict(w: wl.Workload, world: int, graph: bool = False) -> dict:
    return {"workload": w.name, "streams_per_gpu": w.n_streams,
            "new_tokens_per_round": w.new_tokens, "vocab": w.vocab,
            "logits_dtype": w.logits_dtype, "kv_dtype": w.kv_dtype,
            "planes": 2 * w.planes_per_stream, "head_dim": w.head_dim,
            "capacity": w.capacity, "budget": w.budget, "n_sink": w.n_sink,
            "n_recent": w.n_recent, "decay": w.decay, "parallelism": f"streams x{world}",
            "l2": f"inputs larger than L2 (logits rotate through {logits_pool_size(w)} tensors, "
                  f"K/V cache of {2 * w.n_streams * w.planes_per_stream * w.capacity * w.head_dim * 2 >> 20} MiB)",
            "cuda_graph": graph}


def run_ours(args, rank, world, local_rank):
    from paper_2405_12528_b200 import binding as B
    B.lib()                                       # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    w = wl.WORKLOADS[args.workload]
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    p = Pass(w, seed=0, dev=dev, stream_ids=sharding.owned_streams(w.n_streams, rank))
    p.prime()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_rounds(p, rounds=3)

    def sync():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        p.step()
    sync()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graph = None
    if args.graph:       # two rounds (two of the logits tensors) captured once, replayed K/2 times
        assert args.steps % 2 == 0, "--graph needs an even --steps"
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                p.step()
                p.step()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        sync()
    with ClockSampler(local_rank) as clk:
        # the sampler needs a few hundred ms of the same load to see the clocks the timed
        # rounds run at: keep stepping (untimed) before the timed region starts
        soak_end = time.perf_counter() + 0.3
        while time.perf_counter() < soak_end:
            for _ in range(8):
                p.step()
            torch.cuda.synchronize()
        sync()
        t0.record()
        if graph is None:
            for _ in range(args.steps):
                p.step()
        else:
            for _ in range(args.steps // 2):
                graph.replay()
        t1.record()
        sync()
    ms_total = sharding.max_over_ranks(t0.elapsed_time(t1), dev)
    assert B.sirllm_status(p.ws) == 0
    ms_step = ms_total / args.steps
    tokens = world * w.n_streams * w.new_tokens
    value = tokens / (ms_step * 1e-3)

    # per-phase durations of the same rounds (events between the three launches)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    phase_ms, moved = [0.0, 0.0, 0.0], []
    for i in range(args.steps):
        p.step(evs[i])
        torch.cuda.synchronize()
        moved.append(p.moved_rows())
        for j in range(3):
            phase_ms[j] += evs[i][j].elapsed_time(evs[i][j + 1]) / args.steps
    peak, peak_kind = measured_hbm_peak()
    mean_moved = sum(moved) / len(moved)
    by = step_bytes(w, mean_moved)
    compact_gbs = by["compact"] / (phase_ms[2] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "compact_kernel", "achieved": round(compact_gbs, 1),
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": round(compact_gbs / peak, 4),
                "traffic": ncu_traffic(by["compact"]) if w.row_bytes == 256 and w.name != "tiny" else None,
                "traffic_source": "ncu dram bytes of one launch on %s, scaled by moved bytes" % NCU_CAPTURE["workload"],
                "bytes_per_launch": by["compact"], "ms_per_launch": round(phase_ms[2], 4),
                "moved_rows_per_round": mean_moved,
                "phases_ms": {"score": round(phase_ms[0], 4), "select": round(phase_ms[1], 4),
                              "compact": round(phase_ms[2], 4)},
                "score_gbs": round(by["score"] / (phase_ms[0] * 1e-3) / 1e9, 1),
                "step_bytes": by["step"],
                "step_gbs": round(by["step"] / (ms_step * 1e-3) / 1e9, 1),
                "step_frac": round(by["step"] / (ms_step * 1e-3) / 1e9 / peak, 4),
                "step_frac_of_8000": round(by["step"] / (ms_step * 1e-3) / 1e9 / 8000.0, 4)}

    extras = run_extras(p, args) if args.extras else None
    e2e = run_e2e(p, args, dist, world)

    if rank == 0:
        line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_step, 4),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": config_dict(w, world, bool(args.graph)),
                "clocks": clk.result, "e2e": e2e, "gpu_launches": 3 * args.steps,
                "roofline": roofline}
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        if extras is not None:
            line["extras"] = extras
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def _time_rounds(fn, n):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(n):
        fn()
    t1.record()
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / n


def run_extras(p: Pass, args):
    """Timings of the widened entry points on the same state: the fused round fed by per-tile
    (max, sum-exp) pairs instead of logits, and the comparison policies' keep lists + gather."""
    w, B, cfg = p.w, p.B, p.cfg
    tile = 128
    n_tiles = (w.vocab + tile - 1) // tile
    pools = []
    for lg, ids in p.pool[:2]:                   # what an LM-head epilogue would hand over
        rows = lg.shape[0]
        pairs = torch.empty(rows, n_tiles, 2, dtype=torch.float32, device=p.dev)
        for r0 in range(0, rows, 512):
            z = torch.full((min(512, rows - r0), n_tiles * tile), float("-inf"), device=p.dev)
            z[:, :w.vocab] = lg[r0:r0 + 512].float()
            z = z.view(-1, n_tiles, tile)
            m = z.max(dim=2).values
            pairs[r0:r0 + 512, :, 0] = m
            pairs[r0:r0 + 512, :, 1] = torch.exp(z - m[:, :, None]).sum(dim=2)
        target = lg.float()[torch.arange(rows, device=p.dev), ids.long()].contiguous()
        pools.append((pairs, target, ids))
    state = {"i": 0}

    def pairs_round():
        pairs, target, ids = pools[state["i"] & 1]
        state["i"] += 1
        B.sirllm_step_pairs(cfg, pairs, target, ids, p.n_new, p.scores, p.serial, p.live_len, p.decay,
                            p.k, p.v, p.keep_idx, p.n_keep, p.new_entropy, p.ws)

    out = {"pairs_tile": tile,
           "step_pairs_ms": round(_time_rounds(pairs_round, args.steps), 4)}
    if w.head_dim % 16 == 0:
        p.step()                                   # an entropy-selected keep list
        # rotary re-indexing of the K rows the last compaction moved (keep lists of that round)
        ms = _time_rounds(lambda: B.sirllm_rerotate_keys(cfg, p.k, p.keep_idx, p.n_keep, 500000.0,
                                                         B.ROPE_HALF), args.steps)
        moved = p.moved_rows()
        out["rerotate_ms"] = round(ms, 4)
        out["rerotate_gbs"] = round(2 * moved * w.row_bytes * w.planes_per_stream / (ms * 1e-3) / 1e9, 1)
    full = torch.full_like(p.live_len, w.budget + w.new_tokens)
    for name, pol in (("stream", B.POLICY_STREAM), ("random", B.POLICY_RANDOM), ("interval", B.POLICY_INTERVAL)):
        def policy_round():
            state["i"] += 1
            B.sirllm_keep_policy(cfg, pol, full, 7, state["i"], 0, p.keep_idx, p.n_keep, p.ws)
            B.sirllm_compact_kv(cfg, p.k, p.v, p.k, p.v, p.keep_idx, p.n_keep, p.ws)
        out[f"policy_{name}_ms"] = round(_time_rounds(policy_round, args.steps), 4)
    assert B.sirllm_status(p.ws) == 0
    p.live_len.fill_(w.budget)
    return out


def run_e2e(p: Pass, args, dist, world):
    """The same rounds through sirllm_step_host: inputs start in pinned host memory, the
    round's results (keep lists, new lengths, new scores) end in pinned host memory."""
    w, B, cfg = p.w, p.B, p.cfg
    S, P, M, D = w.n_streams, w.planes_per_stream, w.new_tokens, w.head_dim
    pin = lambda t: t.cpu().pin_memory()
    h_pool = [(pin(lg), pin(ids)) for lg, ids in p.pool[:2]]
    serials = torch.arange(M, device=p.dev)
    h_k = torch.empty(S, P, M, D, dtype=w.torch_kv_dtype).pin_memory()
    h_v = torch.empty(S, P, M, D, dtype=w.torch_kv_dtype).pin_memory()
    for s in range(S):
        h_k[s] = wl.make_kv_rows(w, p.seed, "k", p.sid[s], serials, device=p.dev).cpu()
        h_v[s] = wl.make_kv_rows(w, p.seed, "v", p.sid[s], serials, device=p.dev).cpu()
    h_n_new = torch.full((S,), M, dtype=torch.int32).pin_memory()
    h_len = p.live_len.cpu().pin_memory()
    h_keep = torch.zeros(S, cfg.threshold, dtype=torch.int32).pin_memory()
    h_nk = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_e = torch.zeros(S * M, dtype=torch.float32).pin_memory()
    d_logits, d_ids = p.pool[0]
    h2d = sum(t.numel() * t.element_size() for t in (h_pool[0][0], h_pool[0][1], h_k, h_v, h_n_new))
    d2h = sum(t.numel() * t.element_size() for t in (h_keep, h_nk, h_e))

    def one(i):
        lg, ids = h_pool[i & 1]
        B.sirllm_step_host(cfg, lg, ids, h_n_new, h_k, h_v, h_len, d_logits, d_ids, p.n_new,
                           p.scores, p.serial, p.live_len, p.decay, p.k, p.v, p.keep_idx, p.n_keep,
                           p.new_entropy, h_keep, h_nk, h_e, p.ws)
        torch.cuda.current_stream().synchronize()      # the caller reads the results
        h_len.copy_(h_nk)

    n = max(2, min(args.steps, 10))
    for i in range(2):
        one(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(n):
        one(i)
    torch.cuda.synchronize()
    dt = sharding.max_over_ranks(time.perf_counter() - t0, p.dev)
    return {"value": round(world * S * M * n / dt, 1), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": round(dt / n * 1e3, 3), "steps": n,
            "call": "sirllm_step_host"}


# --------------------------------------------------------------------------------------------
# the oracle on the host cores: CPU baseline of the CUDA arm and the reference arm
# --------------------------------------------------------------------------------------------

def host_info() -> dict:
    """The machine the oracle was timed on: logical cores, CPU model, memory."""
    model, ram_gb = None, None
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
        with open("/proc/meminfo") as fh:
            for line in fh:
                if line.startswith("MemTotal"):
                    ram_gb = round(int(line.split()[1]) / 2 ** 20, 1)
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu_model": model, "ram_gb": ram_gb}


def oracle_rounds(p: Pass, rounds: int):
    """Times `rounds` full evicting rounds of the oracle, as it stands, on a host copy of the
    device state (1 thread)."""
    import oracle
    w = p.w
    S, M = w.n_streams, w.new_tokens
    p.append_rows()
    torch.cuda.synchronize()
    lg, ids = p.pool[0]
    h_lg, h_ids = lg.cpu(), ids.cpu()
    streams = []
    for s in range(S):
        st = oracle.Stream(w.capacity, w.n_sink, w.n_recent, w.budget, w.threshold, float(p.decay[s]),
                           p.k[s].cpu(), p.v[s].cpu())
        st.E.copy_(p.scores[s].cpu())
        st.live_len = int(p.live_len[s])
        streams.append(st)
    t0 = time.perf_counter()
    for _ in range(rounds):
        for s, st in enumerate(streams):
            e = oracle.score(h_lg[s * M:(s + 1) * M], h_ids[s * M:(s + 1) * M])
            st.step(e)
    dt = time.perf_counter() - t0
    return {"value": round(rounds * S * M / dt, 1), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{rounds} full evicting rounds of {w.name} (all {S * M} tokens, all "
                      f"{2 * w.planes_per_stream * S} planes), {dt:.1f} s of CPU time",
            "seconds_per_round": round(dt / rounds, 3), "host": host_info()}


def run_reference(args, rank, world):
    """The oracle, as it stands, on the host cores: the same workload, metric and unit."""
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = wl.WORKLOADS[args.workload]
    # a bounded slice of the round: a fraction f of the new tokens and of the K/V planes
    # (the pass is linear in both), so that K + W steps end within a few minutes
    full_round_s = (w.n_streams * w.new_tokens * w.vocab / 1.4e8
                    + 4 * w.n_streams * w.planes_per_stream * w.budget * w.row_bytes / 2.0e9)
    f = 1.0
    while f > 1 / 64 and full_round_s * f * (args.steps + args.warmup) > 120.0:
        f /= 2
    if w.n_streams > 1:      # whole streams first, then a slice of each
        S = max(1, int(w.n_streams * f))
        f = min(1.0, f * w.n_streams / S)
    else:
        S = 1
    T = max(1, int(w.new_tokens * f))
    P = max(1, int(w.planes_per_stream * f))
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    bias = wl.zipf_bias_table(w.vocab, w.zipf_bias, dev) if w.zipf_bias else None
    planes = torch.arange(P)
    streams, inputs = [], []
    for s in range(S):
        k = torch.zeros(P, w.capacity, w.head_dim, dtype=w.torch_kv_dtype)
        v = torch.zeros_like(k)
        st = oracle.Stream(w.capacity, w.n_sink, w.n_recent, w.budget, w.threshold,
                           float(wl.stream_decay(w, 0)[s]), k, v)
        first = torch.arange(w.budget)
        k[:, :w.budget] = wl.make_kv_rows(w, 0, "k", s, first, planes, dev).cpu()
        v[:, :w.budget] = wl.make_kv_rows(w, 0, "v", s, first, planes, dev).cpu()
        st.E[:w.budget] = wl.random_scores(s, w.budget)
        st.live_len = w.budget
        st.next_serial.value = w.budget
        streams.append(st)
        inputs.append((wl.make_logits(w, 0, s, 0, T, dev, bias).cpu(),
                       wl.make_token_ids(w, 0, s, 0, T, dev).cpu()))

    def one():
        for st, (lg, ids) in zip(streams, inputs):
            e = oracle.score(lg, ids)
            pad = torch.zeros(w.new_tokens - T)      # the rest of the round's tokens: score 0
            st.step(torch.cat([e, pad]))

    for _ in range(args.warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one()
    dt = (time.perf_counter() - t0) / args.steps
    value = S * T / dt
    sample = (f"per step: {S} of {w.n_streams} streams, {T} of {w.new_tokens} new tokens scored and "
              f"{2 * P} of {2 * w.planes_per_stream} K/V planes compacted per stream (the same "
              f"fraction of both; selection over the full cache)")
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 1), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, world),
            "cpu_baseline": {"value": round(value, 1), "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": sample, "host": host_info()},
            "e2e": {"value": round(value, 1), "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def launch_ranks(n: int) -> int:
    """Started plainly with --gpus N: run N copies of this script as ranks 0..N-1, one per GPU
    (the environment torchrun would have set, rendezvous on 127.0.0.1), and wait for them.
    Rank 0 prints the job's line on the inherited stdout."""
    visible = torch.cuda.device_count()
    if n > visible:
        print(f"bench.py: --gpus {n} needs {n} visible CUDA devices, this machine shows {visible}; "
              f"nothing was run", file=sys.stderr)
        return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], env=env))
    rc = 0
    for proc in procs:
        rc = max(rc, abs(proc.wait()))
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(wl.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extras", action="store_true",
                    help="also time the pairs-fed round and the comparison policies")
    ap.add_argument("--graph", action="store_true",
                    help="replay the timed rounds from a captured CUDA graph (launch-bound shapes)")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    under_launcher = "WORLD_SIZE" in os.environ
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if under_launcher and world != args.gpus and rank == 0:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks; reporting "
              f"n_gpus = {world}", file=sys.stderr)
    if args.impl == "reference":
        # the oracle runs on the host cores of rank 0 alone, whatever N is
        run_reference(args, rank, world if under_launcher else args.gpus)
    elif not under_launcher and args.gpus > 1:
        sys.exit(launch_ranks(args.gpus))
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
