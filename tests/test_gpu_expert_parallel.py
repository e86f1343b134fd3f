"""The expert-parallel layer with the library's kernels: two ranks as two processes sharing the one
GPU, exchanging over gloo (host-synchronised collectives: no kernel of one rank waits for a kernel of
the other).  Each rank holds half of the tokens and half of the experts and compares its shard of
every output with the single-device layer run on the whole batch in the same process."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from gen import workloads as gw
        from paper_2406_00023_b200 import etr, expert_parallel as ep
        torch.cuda.set_device(0)
        w = gw.scaled(gw.WORKLOADS["mid"], T=1024, d=512, D=8, E=8, h=256, n_clusters=8)
        inp = gw.make_inputs(w)
        bf = torch.bfloat16
        X, dY, W1g, W1u, W2 = (torch.from_numpy(inp[k]).to(bf).cuda() for k in ("X", "dY", "W1g", "W1u", "W2"))
        R = torch.from_numpy(inp["R"]).cuda()
        # single-device reference on the whole batch
        cfg = etr.make_config(T=w.T, d=w.d, D=w.D, E=w.E, k=w.k, h=w.h, capacity=w.capacity, dtype=etr.BF16,
                              mode=etr.MODE_ECR)
        buf = etr.LayerBuffers(cfg)
        ref = dict(Y=torch.empty_like(X), dX=torch.empty_like(X), dR=torch.empty_like(R),
                   dW1g=torch.empty_like(W1g), dW1u=torch.empty_like(W1u), dW2=torch.empty_like(W2))
        etr.layer_forward(cfg, X, R, W1g, W1u, W2, buf, ref["Y"])
        etr.layer_backward(cfg, X, R, W1g, W1u, W2, dY, buf, ref["dX"], ref["dR"], ref["dW1g"], ref["dW1u"],
                           ref["dW2"])
        torch.cuda.synchronize()
        # this rank's shard through the expert-parallel layer
        Tl, El = w.T // world, w.E // world
        tok, exp = slice(rank * Tl, (rank + 1) * Tl), slice(rank * El, (rank + 1) * El)
        layer = ep.ExpertParallelLayer(T_local=Tl, d=w.d, D=w.D, E=w.E, h=w.h, capacity=w.capacity)
        Xl, dYl = X[tok].contiguous(), dY[tok].contiguous()
        Wl = [t[exp].contiguous() for t in (W1g, W1u, W2)]
        Y = layer.forward(Xl, R, *Wl)
        dX, dR, dW1g, dW1u, dW2 = layer.backward(Xl, R, *Wl, dYl)
        torch.cuda.synchronize()
        Cs = etr.c_stride(cfg)
        rows = slice(rank * El * Cs, (rank + 1) * El * Cs)
        # routing of the local experts over all tokens, and everything the local GEMMs produce: identical
        assert torch.equal(layer.own.slot_token, buf.slot_token[rows])
        assert torch.equal(layer.own.gate, buf.gate[rows])
        assert float(layer.delta_max) == buf.read_stats().delta_max
        for nm in ("Xp", "G", "U", "H", "O", "dO", "dG", "dU", "dXp"):
            assert torch.equal(getattr(layer.own, nm), getattr(buf, nm)[rows]), nm
        for got, nm in ((dW1g, "dW1g"), (dW1u, "dW1u"), (dW2, "dW2")):
            assert torch.equal(got, ref[nm][exp]), nm

        def close(a, b, ulps, rel, what):
            a, b = a.float(), b.float()
            rms = b.pow(2).mean().sqrt()
            assert bool(((a - b).abs() <= ulps * 2.0 ** -7 * b.abs() + rel * rms).all()), what

        # Y: the same products summed with a multiply and an add instead of a fused multiply-add
        close(Y, ref["Y"][tok], 1, 1e-3, "Y")
        # dX: the sum of the token's rows of dXp is rounded to bf16 before the router term is added (the
        # single-device layer keeps it in fp32): one more rounding of a sum that may cancel
        close(dX, ref["dX"][tok], 2, 1e-2, "dX")
        unrouted = torch.from_numpy(np.diff(buf.tok_ptr.cpu().numpy())[tok] == 0).cuda()
        assert bool((Y[unrouted] == 0).all()) and bool((dX[unrouted] == 0).all()) and int(unrouted.sum()) > 0
        rel = (dR - ref["dR"]).abs().max() / ref["dR"].pow(2).mean().sqrt()
        assert float(rel) < 1e-4, ("dR", float(rel))
        q.put((rank, "ok"))
    except Exception as e:      # report instead of leaving the peer in a collective
        q.put((rank, f"{type(e).__name__}: {e}"))
        raise
    finally:
        dist.destroy_process_group()


def test_expert_parallel_layer_on_two_ranks_sharing_the_gpu():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
    assert [r[1] for r in res] == ["ok", "ok"], res
