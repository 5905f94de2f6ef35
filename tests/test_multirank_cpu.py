"""Host logic of the multi-GPU path on CPU ranks (gloo, world size 2): the batch is sharded by sequence with no
data-path exchange; the only collective is the max-over-ranks of the step time that the benchmark reports."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_16439_b200 import workloads as wl


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, B_total: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = wl.shard_batch(B_total, rank, world)
        # every rank draws its own sequences (seed offset by rank, as the benchmark does) and would run them alone
        shape = wl.Shape("shard", 1, hi - lo, 4, 2, 128, 4, 1, 3, 1, "f32")
        p = wl.decode_inputs(shape, 7, wl.layer_seed(0, 0) + 100000 * rank, "cpu")
        owned = torch.zeros(B_total, dtype=torch.int32)
        owned[lo:hi] = 1
        dist.all_reduce(owned, op=dist.ReduceOp.SUM)              # test-only: every sequence has exactly one owner
        t = torch.tensor([10.0 + rank])                           # this rank's step time in ms
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
        out.put((rank, lo, hi, owned.tolist(), float(t.item()), float(p["q"].sum())))
    finally:
        dist.destroy_process_group()


def test_batch_sharding_and_max_over_ranks_timing_with_two_gloo_ranks():
    world, B_total = 2, 9
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, B_total, out)) for r in range(world)]
    for pr in procs:
        pr.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    (r0, lo0, hi0, owned0, t0, s0), (r1, lo1, hi1, owned1, t1, s1) = res
    assert (lo0, hi0, lo1, hi1) == (0, 5, 5, 9)                   # contiguous, disjoint, the remainder goes to the first ranks
    assert owned0 == owned1 == [1] * B_total
    assert t0 == t1 == 11.0                                       # the slowest rank's time is the step time on every rank
    assert s0 != s1                                               # ranks draw different sequences
    # aggregate throughput as the benchmark reports it: all ranks' sequences over the max time
    steps = 4
    assert abs(B_total * steps / (t0 * 1e-3) - (5 + 4) * steps / 11e-3) < 1e-6


def test_shard_batch_covers_every_split():
    for B in (1, 2, 7, 8, 64):
        for world in (1, 2, 3, 8):
            spans = [wl.shard_batch(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
