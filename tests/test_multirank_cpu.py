"""The N > 1 host logic on CPU: two gloo ranks agree on a disjoint, complete and balanced
split of a model's tensors without talking to each other, and timings reduce to the
slowest rank's.  No kernel runs here."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads
from paper_2505_02380_b200 import multirank


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _chunk_counts(wl):
    return [(t.numel + wl.chunk_symbols - 1) // wl.chunk_symbols for t in wl.tensors]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = workloads.mistral_7b(bits=8)
        counts = _chunk_counts(wl)
        mine = multirank.shard_tensors(counts, world)[rank]
        # every rank tells the others what it took (test-only exchange)
        got = [None] * world
        dist.all_gather_object(got, mine)
        slowest = multirank.max_over_ranks(10.0 + rank)
        total = multirank.sum_over_ranks(float(sum(counts[i] for i in mine)))
        q.put((rank, got, slowest, total, sum(counts)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = workloads.mistral_7b(bits=8)
    counts = _chunk_counts(wl)
    for rank, got, slowest, total, all_chunks in res:
        assert slowest == 11.0                       # max over ranks
        assert total == float(all_chunks)            # the shards cover every chunk exactly once
        flat = sorted(i for part in got for i in part)
        assert flat == list(range(len(counts)))      # disjoint and complete
        loads = [sum(counts[i] for i in part) for part in got]
        assert max(loads) - min(loads) <= max(counts)  # balanced to within one tensor


def test_shard_is_deterministic_and_handles_edge_cases():
    assert multirank.shard_tensors([], 3) == [[], [], []]
    assert multirank.shard_tensors([5], 2) == [[0], []]
    a = multirank.shard_tensors([7, 7, 7, 7, 1, 1], 2)
    assert a == multirank.shard_tensors([7, 7, 7, 7, 1, 1], 2)
    assert sorted(a[0] + a[1]) == list(range(6))
    assert abs(sum([7, 7, 7, 7, 1, 1][i] for i in a[0]) - 15) <= 1
    assert multirank.max_over_ranks(3.5) == 3.5      # no process group: identity
