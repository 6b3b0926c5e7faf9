"""World-size-2 run of the multi-GPU plumbing on CPU (gloo): streams shard across ranks with
no data-path collective; only timings and counts are reduced."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2405_12528_b200 import sharding
from paper_2405_12528_b200 import workloads as wl


def test_stream_ownership_is_a_partition():
    for world in (1, 2, 3, 8):
        ids = [i for r in range(world) for i in sharding.owned_streams(5, r)]
        assert ids == list(range(5 * world))
        for total in (1, 7, 64):
            parts = [sharding.split_streams(total, world, r) for r in range(world)]
            assert [i for p in parts for i in p] == list(range(total))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _one_round_on_the_oracle(w, stream_id):
    """One evicting round of one stream, computed by the oracle (stand-in for a GPU)."""
    st = oracle.Stream(w.capacity, w.n_sink, w.n_recent, w.budget, w.threshold, w.decay)
    logits = wl.make_logits(w, 0, stream_id, 0)
    ids = wl.make_token_ids(w, 0, stream_id, 0)
    keep = st.step(oracle.score(logits, ids))
    return keep


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.WORKLOADS["tiny"].scaled(new_tokens=96, budget=64, n_recent=16, vocab=997, capacity=128)
        mine = sharding.owned_streams(2, rank)
        digests = []
        for sid in mine:                                    # no communication on the data path
            keep = _one_round_on_the_oracle(w, sid)
            digests.append(int(keep.long().sum()))
        gathered = [None] * world
        dist.all_gather_object(gathered, (list(mine), digests))
        slowest = sharding.max_over_ranks(1.5 * (rank + 1))
        tokens = sharding.sum_over_ranks(len(mine) * w.new_tokens)
        out.put((rank, gathered, slowest, tokens))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_streams_and_reduce_only_bookkeeping():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = wl.WORKLOADS["tiny"].scaled(new_tokens=96, budget=64, n_recent=16, vocab=997, capacity=128)
    single = [int(_one_round_on_the_oracle(w, sid).long().sum()) for sid in range(4)]
    for rank, gathered, slowest, tokens in results:
        ids = [i for owned, _ in gathered for i in owned]
        got = [d for _, dig in gathered for d in dig]
        assert ids == [0, 1, 2, 3]                      # every stream owned exactly once
        assert got == single                            # sharded result == single-process result
        assert len(set(single)) > 1                     # and the streams really differ
        assert slowest == 3.0                           # max over ranks
        assert tokens == 4 * 96                         # whole-job count


# ---- vocabulary-parallel scoring: the exchange, with the oracle standing in for the GPUs ----

def _vocab_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.WORKLOADS["tiny"].scaled(new_tokens=40, vocab=1001)
        logits = wl.make_logits(w, 0, 0, 0)
        ids = wl.make_token_ids(w, 0, 0, 0)
        ids[3] = -1
        v0, v1 = sharding.vocab_ranges(w.vocab, world)[rank]
        # this rank only ever looks at its own columns
        pairs_local, target_local = oracle.range_pairs(logits[:, v0:v1].contiguous(), ids - v0 * (ids >= 0),
                                                       0, v1 - v0)
        pairs, target = sharding.exchange_vocab_partials(pairs_local, target_local)
        e = oracle.score_pairs(pairs, target, ids, w.vocab)
        out.put((rank, tuple(pairs.shape), e.tolist()))
    finally:
        dist.destroy_process_group()


def test_vocab_ranges_cover_the_vocabulary():
    for vocab, world in ((32000, 8), (128256, 3), (5, 8), (1001, 2)):
        r = sharding.vocab_ranges(vocab, world)
        assert r[0][0] == 0 and r[-1][1] == vocab and len(r) == world
        assert all(a[1] == b[0] for a, b in zip(r[:-1], r[1:]))
        assert max(b - a for a, b in r) - min(b - a for a, b in r) <= 1


def test_two_ranks_score_a_vocabulary_split_across_them():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_vocab_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = wl.WORKLOADS["tiny"].scaled(new_tokens=40, vocab=1001)
    ids = wl.make_token_ids(w, 0, 0, 0)
    ids[3] = -1
    want = oracle.score(wl.make_logits(w, 0, 0, 0), ids)
    for rank, shape, e in results:
        assert shape == (40, 2, 2)
        assert e == results[0][2]                         # every rank ends with the same scores
        assert torch.allclose(torch.tensor(e), want, rtol=0, atol=2e-6)
        assert e[3] == 0.0


def test_plane_shards_partition_the_planes():
    for by, (L, H) in (("layers", (32, 8)), ("heads", (32, 8)), ("layers", (5, 3))):
        for world in (1, 2, 4):
            owned = [sharding.plane_shard(L, H, world, r, by) for r in range(world)]
            planes = sorted((l, h) for ls, hs in owned for l in ls for h in hs)
            assert planes == [(l, h) for l in range(L) for h in range(H)]
