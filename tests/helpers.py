"""Shared test plumbing: device state of a workload and its oracle twin."""
from __future__ import annotations

import torch

import oracle
from paper_2405_12528_b200 import binding as B
from paper_2405_12528_b200 import workloads as wl

ENTROPY_ABS, ENTROPY_REL = 1e-5, 1e-4


def assert_entropy_close(got: torch.Tensor, want: torch.Tensor):
    """|g - o| <= max(1e-5, 1e-4 * |o|): fp32 accumulation against the fp64 oracle."""
    got, want = got.double().cpu(), want.double().cpu()
    tol = torch.clamp(ENTROPY_REL * want.abs(), min=ENTROPY_ABS)
    bad = (got - want).abs() > tol
    assert not bad.any(), (f"{int(bad.sum())} scores out of tolerance; worst "
                           f"{float(((got - want).abs() / tol).max()):.2f} x tol")


class DeviceState:
    """Device buffers of a workload (all streams) for the C-ABI calls."""

    def __init__(self, w: wl.Workload, seed: int = 0, device="cuda", with_kv=True, **cfg_over):
        self.w, self.seed, self.dev = w, seed, device
        self.cfg = B.config_from_workload(w, **cfg_over)
        S, P, C, D = w.n_streams, w.planes_per_stream, self.cfg.capacity, w.head_dim
        self.ws = B.new_workspace(self.cfg, device)
        self.scores = torch.zeros(S, C, dtype=torch.float32, device=device)
        self.serial = torch.full((S, C), -1, dtype=torch.int64, device=device)
        self.live_len = torch.zeros(S, dtype=torch.int32, device=device)
        self.decay = wl.stream_decay(w, seed).to(device)
        self.keep_idx = torch.full((S, self.cfg.threshold), -1, dtype=torch.int32, device=device)
        self.n_keep = torch.zeros(S, dtype=torch.int32, device=device)
        self.new_entropy = torch.zeros(S * self.cfg.max_new, dtype=torch.float32, device=device)
        self.k = self.v = None
        if with_kv:
            self.k = torch.zeros(S, P, C, D, dtype=w.torch_kv_dtype, device=device)
            self.v = torch.zeros(S, P, C, D, dtype=w.torch_kv_dtype, device=device)
        self.logits = torch.zeros(S * self.cfg.max_new, w.vocab, dtype=w.torch_logits_dtype, device=device)
        self.token_ids = torch.zeros(S * self.cfg.max_new, dtype=torch.int32, device=device)
        self.n_new = torch.zeros(S, dtype=torch.int32, device=device)
        self.next_serial = [0] * S
        self.host_len = [0] * S
        self.bias = wl.zipf_bias_table(w.vocab, w.zipf_bias, device) if w.zipf_bias else None

    def fill_round(self, rnd: int, n_new=None, rho=None):
        """Generate the round's logits / ids on the device and write the new K/V rows and
        serial tags into slots [live_len, live_len + n_new) of every plane."""
        w, M = self.w, self.cfg.max_new
        n_new = [w.new_tokens] * w.n_streams if n_new is None else list(n_new)
        for s in range(w.n_streams):
            T, l = n_new[s], self.host_len[s]
            wl.make_logits(w, self.seed, s, rnd, T, self.dev, self.bias, out=self.logits[s * M:s * M + T])
            self.token_ids[s * M:s * M + T] = wl.make_token_ids(w, self.seed, s, rnd, T, self.dev, rho)
            serials = torch.arange(self.next_serial[s], self.next_serial[s] + T, device=self.dev)
            if l + T <= self.cfg.capacity:
                self.serial[s, l:l + T] = serials
                if self.k is not None:
                    self.k[s, :, l:l + T] = wl.make_kv_rows(w, self.seed, "k", s, serials, device=self.dev)
                    self.v[s, :, l:l + T] = wl.make_kv_rows(w, self.seed, "v", s, serials, device=self.dev)
                self.next_serial[s] += T
        self.n_new.copy_(torch.tensor(n_new, dtype=torch.int32))
        return n_new

    def enqueue_step(self):
        B.sirllm_step(self.cfg, self.logits, self.token_ids, self.n_new, self.scores, self.serial,
                      self.live_len, self.decay, self.k, self.v, self.keep_idx, self.n_keep,
                      self.new_entropy, self.ws)

    def step(self):
        self.enqueue_step()
        self.host_len = self.live_len.cpu().tolist()

    def check_kv_by_content(self, streams=None):
        """Every live K/V row must be the row of the token whose serial tag sits in its slot."""
        w = self.w
        for s in (range(w.n_streams) if streams is None else streams):
            n = self.host_len[s]
            live = self.serial[s, :n]
            assert torch.equal(self.k[s, :, :n], wl.make_kv_rows(w, self.seed, "k", s, live, device=self.dev))
            assert torch.equal(self.v[s, :, :n], wl.make_kv_rows(w, self.seed, "v", s, live, device=self.dev))


def oracle_twin(w: wl.Workload, decay, with_kv=True, threshold=None):
    """One oracle stream per device stream (CPU copies of the caches)."""
    out = []
    for s in range(w.n_streams):
        k = v = None
        if with_kv:
            k = torch.zeros(w.planes_per_stream, w.capacity, w.head_dim, dtype=w.torch_kv_dtype)
            v = torch.zeros_like(k)
        out.append(oracle.Stream(w.capacity, w.n_sink, w.n_recent, w.budget,
                                 w.threshold if threshold is None else threshold,
                                 float(decay[s]), k, v))
    return out
