"""Expert-parallel exchange (paper_2406_00023_b200/expert_parallel.py) on two gloo ranks, CPU only.

Each rank holds half of the tokens and half of the experts.  The per-rank arithmetic is the oracle's
(this is a test of the exchange plan, not of the kernels); every exchanged quantity is compared with
the single-process oracle run on the whole batch: the affinity columns and batch maximum an owner
receives, the selection it takes over all tokens, the rows that land in its experts' buffers, the
combined outputs every token holder ends with, and the two exchanges of the backward pass."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

T, E, D, d, h, K, C = 96, 4, 4, 32, 16, 2, 20


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem():
    from gen import workloads as gw
    w = gw.scaled(gw.WORKLOADS["mid"], T=T, d=d, D=D, E=E, h=h, n_clusters=4, dtype="f32", cf=C * E / (T * K))
    assert w.capacity == C
    return w, gw.make_inputs(w)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import binding as ob
        from paper_2406_00023_b200 import expert_parallel as ep
        ob.set_threads(1)
        o = ob.Oracle("f64")
        w, inp = _problem()
        X, R, dY = (inp[k].astype(np.float64) for k in ("X", "R", "dY"))
        W1g, W1u, W2 = (inp[k].astype(np.float64) for k in ("W1g", "W1u", "W2"))
        Cs = w.C_stride
        # the single-process reference on the whole batch
        fw = o.forward(X, R, W1g, W1u, W2, D=D, k=K, capacity=C, mode=ob.MODE_ECR)
        bw = o.backward(fw, X, R, W1g, W1u, W2, dY)
        # this rank's shard
        Tl, El = T // world, E // world
        tok = slice(rank * Tl, (rank + 1) * Tl)
        exp = slice(rank * El, (rank + 1) * El)
        rows = slice(rank * El * Cs, (rank + 1) * El * Cs)
        t = torch.from_numpy
        # 1-2. local affinities, then the owners' columns and the batch maximum
        delta_l, xnorm_l, rnorm, _ = o.affinity(X[tok], R, D)
        delta_own, dmax = ep.exchange_affinities(t(delta_l))
        assert np.array_equal(delta_own.numpy(), fw.delta[:, exp]) and float(dmax) == float(fw.delta_max)
        # 3. selection for the local experts over all tokens
        rt = o.select(delta_own.numpy(), K, ob.MODE_ECR, C, Cs)
        assert np.array_equal(rt.slot_token, fw.route.slot_token[rows])
        assert np.array_equal(rt.gate, fw.route.gate[rows])
        # 4-5. plan and the forward row exchange
        plan = ep.build_plan(t(rt.slot_token), t(rt.gate), Tl)
        assert sum(plan.rows_in) == int(rt.counts.sum()) <= El * C
        Xp = ep.dispatch_rows(plan, t(np.ascontiguousarray(X[tok])), El * Cs)
        assert np.array_equal(Xp.numpy(), fw.Xp[rows])
        # 6. local experts
        G, U, H, O = o.expert_ffn(Xp.numpy(), rt, W1g[exp], W1u[exp], W2[exp])
        assert np.array_equal(O, fw.O[rows])
        # 7. rows back and the combine, in ascending expert order
        back = ep.return_rows(plan, t(O))
        Y = ep.combine_local(plan, back, torch.float64)
        assert np.allclose(Y.numpy(), fw.Y[tok], rtol=1e-14, atol=1e-300)
        unrouted = np.diff(fw.route.tok_ptr)[tok] == 0
        assert np.all(Y.numpy()[unrouted] == 0)
        # backward: d O = gate * dY goes out in the plan's order, d Xp comes back and is summed per token
        send_tok = torch.cat(plan.send_tokens)
        dO_rows = t(np.ascontiguousarray(dY[tok]))[send_tok] * torch.cat(plan.send_gates)[:, None]
        dO = ep.scatter_rows_to_experts(plan, dO_rows, El * Cs)
        assert np.allclose(dO.numpy(), bw.dO[rows], rtol=1e-15, atol=0)
        dgate_rows = (t(np.ascontiguousarray(dY[tok]))[send_tok] * back).sum(1, keepdim=True)   # <dY[t], O[r]>
        dgate = ep.scatter_rows_to_experts(plan, dgate_rows, El * Cs)[:, 0]
        assert np.allclose(dgate.numpy(), bw.dgate[rows], rtol=1e-12, atol=1e-300)
        dXp_back = ep.return_rows(plan, t(np.ascontiguousarray(bw.dXp[rows])))
        for qq in range(world):          # the token side knows which buffer row each of its rows fills
            own_rows = np.arange(qq * El * Cs, (qq + 1) * El * Cs)[plan.send_rows[qq].numpy()]
            assert np.array_equal(fw.route.slot_token[own_rows], plan.send_tokens[qq].numpy() + rank * Tl)
        ones = ep.with_unit_gates(plan)
        dX_ffn = ep.combine_local(ones, dXp_back, torch.float64)
        assert np.allclose(dX_ffn.numpy(), bw.dX_ffn[tok], rtol=1e-14, atol=1e-300)
        q.put((rank, "ok", sum(plan.rows_in), sum(plan.rows_out)))
    except Exception as e:      # report instead of hanging the peer's collective
        q.put((rank, f"{type(e).__name__}: {e}", 0, 0))
        raise
    finally:
        dist.destroy_process_group()


def test_exchange_plan_matches_the_single_process_oracle_on_two_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
    assert [r[1] for r in res] == ["ok", "ok"], res
    assert sum(r[2] for r in res) == sum(r[3] for r in res) == E * C       # expert choice fills every expert
