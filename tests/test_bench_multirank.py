"""Host-side logic of the multi-GPU benchmark path, run as two gloo ranks on the CPU.

With N > 1 the benchmark runs N independent replicas (the layer has no exchange step); the
only cross-rank operations are the barrier and the max-over-ranks of the device timings.
"""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from dataclasses import replace
    from gen import workloads as gw
    # each replica draws its own tokens
    w = replace(gw.WORKLOADS["tiny"], config_id=gw.WORKLOADS["tiny"].config_id + 1000 * rank)
    x = gw.tokens(w)
    dist.barrier()
    ms = bench.aggregate_over_ranks([10.0 + 5.0 * rank, 3.0 - rank], world)
    q.put((rank, ms, float(x[0, 0]), bench.whole_job_tokens_per_sec(world, w.T, ms[0])))
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_rank_and_sum_the_tokens():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, x0, v0), (r1, ms1, x1, v1) = res
    assert ms0 == ms1 == [15.0, 3.0]                 # element-wise max over the ranks
    assert x0 != x1                                  # replicas see different tokens
    assert v0 == v1 == 2 * 512 / 15e-3               # whole-job tokens/s: all ranks' tokens


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.aggregate_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
