"""Pins for the oracle's FFN / combine half and for every gradient.

Forward: library SwiGLU (torch float64) for one expert and for the dense reduction
(expert choice with C = T selects every pair, so Y[t] = sum_i delta_ti E_i(x_t)), the
dispatch/CSR identity, permutation equivariance.  Backward: central finite differences
of the double-precision oracle with the selection frozen, torch.autograd of the dense
reduction, and the orthogonality identities that scale invariance of the cosine forces.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from gen import workloads as gw
from oracle import binding as ob


@pytest.fixture(scope="module")
def o32():
    return ob.Oracle("f32")


@pytest.fixture(scope="module")
def o64():
    return ob.Oracle("f64")


def problem(seed, T=12, d=8, D=2, E=3, h=6):
    rng = np.random.default_rng(seed)
    q, _ = np.linalg.qr(rng.standard_normal((d // D, E)))
    return dict(X=rng.standard_normal((T, d)), R=q.T.copy(),
                W1g=rng.standard_normal((E, h, d)) / np.sqrt(d),
                W1u=rng.standard_normal((E, h, d)) / np.sqrt(d),
                W2=rng.standard_normal((E, d, h)) / np.sqrt(d),
                dY=rng.standard_normal((T, d)))


def torch_swiglu(x, W1g, W1u, W2):
    return (F.silu(x @ W1g.T) * (x @ W1u.T)) @ W2.T


def torch_affinity(X, R, D):
    """cos(x_t, w_i) with w_i the dense d-vector of the GrAP router (library ops only)."""
    W = R.repeat_interleave(D, dim=1) / D
    return F.cosine_similarity(X[:, None, :], W[None, :, :], dim=-1, eps=0.0)


def test_single_expert_is_library_swiglu(o64):
    p = problem(1, E=1, D=2)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=1, capacity=12,
                     mode=ob.MODE_TCR)
    t = {k: torch.from_numpy(v) for k, v in p.items()}
    ref = torch_affinity(t["X"], t["R"], 2) * torch_swiglu(t["X"], t["W1g"][0], t["W1u"][0], t["W2"][0])
    assert np.allclose(fw.Y, ref.numpy(), rtol=1e-12, atol=1e-13)
    assert fw.route.counts.tolist() == [12]


def dense_moe_torch(t, D):
    delta = torch_affinity(t["X"], t["R"], D)
    Y = 0
    for i in range(t["R"].shape[0]):
        Y = Y + delta[:, i:i + 1] * torch_swiglu(t["X"], t["W1g"][i], t["W1u"][i], t["W2"][i])
    return Y


def test_expert_choice_full_capacity_is_dense_moe_fwd_bwd(o64):
    """C = T in expert choice: the general MoE form with every gate active.  Forward and
    all five gradients against torch.autograd in float64."""
    p = problem(2)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=12,
                     mode=ob.MODE_ECR)
    bw = o64.backward(fw, p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], p["dY"])
    t = {k: torch.from_numpy(v).requires_grad_(k != "dY") for k, v in p.items()}
    Y = dense_moe_torch(t, 2)
    (Y * t["dY"]).sum().backward()
    assert np.allclose(fw.Y, Y.detach().numpy(), rtol=1e-12, atol=1e-13)
    for name, got in [("X", bw.dX), ("R", bw.dR), ("W1g", bw.dW1g), ("W1u", bw.dW1u), ("W2", bw.dW2)]:
        want = t[name].grad.numpy()
        assert np.allclose(got, want, rtol=1e-10, atol=1e-12), name


def test_dispatch_then_inverse_is_identity(o32):
    w = gw.WORKLOADS["tiny"]
    R = gw.expert_embeddings(w)
    X = gw.tokens(w, R)
    delta, *_ = o32.affinity(X, R, D=w.D)
    rt = o32.select(delta, w.k, ob.MODE_TCR, w.capacity, w.C_stride)
    Xp = o32.dispatch(X, rt)
    valid = rt.slot_token >= 0
    assert np.array_equal(Xp[valid], X[rt.slot_token[valid]]) and np.all(Xp[~valid] == 0)
    back = o32.dispatch_bwd(Xp, rt)           # sums the rows of each token
    nrows = np.diff(rt.tok_ptr)[:, None]
    assert np.allclose(back, nrows * X, rtol=1e-6, atol=1e-6)


def test_combine_weights_are_selected_affinities(o32):
    w = gw.WORKLOADS["tiny"]
    R = gw.expert_embeddings(w)
    X = gw.tokens(w, R)
    delta, *_ = o32.affinity(X, R, D=w.D)
    rt = o32.select(delta, w.k, ob.MODE_TCR, 100, w.C_stride)
    O = np.ones((w.E * w.C_stride, 4), np.float32)      # combine then returns sum of gates
    Y = o32.combine(O, rt)
    want = np.zeros(w.T)
    for r in np.nonzero(rt.slot_token >= 0)[0]:
        want[rt.slot_token[r]] += float(delta[rt.slot_token[r], r // w.C_stride])
    assert np.allclose(Y[:, 0], want, atol=1e-6)
    unrouted = np.diff(rt.tok_ptr) == 0
    assert unrouted.any() and np.all(Y[unrouted] == 0)


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
def test_permutation_equivariance(o64, mode):
    p = problem(3, T=16)
    kw = dict(D=2, k=2, capacity=7, mode=mode)
    base = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], **kw).Y
    perm = np.random.default_rng(0).permutation(16)
    Yp = o64.forward(p["X"][perm], p["R"], p["W1g"], p["W1u"], p["W2"], **kw).Y
    assert np.allclose(Yp, base[perm], atol=1e-13)
    ep = np.array([2, 0, 1])
    Ye = o64.forward(p["X"], p["R"][ep], p["W1g"][ep], p["W1u"][ep], p["W2"][ep], **kw).Y
    assert np.allclose(Ye, base, atol=1e-13)


@pytest.mark.parametrize("mode,cap", [(ob.MODE_TCR, 5), (ob.MODE_ECR, 5), (ob.MODE_TCR, 3)])
def test_gradients_by_finite_differences(o64, mode, cap):
    p = problem(4)
    kw = dict(D=2, k=2, capacity=cap, mode=mode)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], **kw)
    assert fw.route.dropped > 0                       # the capacity bound is active
    bw = o64.backward(fw, p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], p["dY"])

    def loss(q):
        y = o64.forward(q["X"], q["R"], q["W1g"], q["W1u"], q["W2"], route=fw.route, **kw).Y
        return float((y * p["dY"]).sum())

    eps = 1e-6
    grads = dict(X=bw.dX, R=bw.dR, W1g=bw.dW1g, W1u=bw.dW1u, W2=bw.dW2)
    rng = np.random.default_rng(5)
    for name, g in grads.items():
        flat_n = p[name].size
        picks = range(flat_n) if flat_n <= 128 else rng.choice(flat_n, 96, replace=False)
        scale = np.abs(g).max()
        for idx in picks:
            q = {k: v.copy() for k, v in p.items()}
            q[name].reshape(-1)[idx] += eps
            up = loss(q)
            q[name].reshape(-1)[idx] -= 2 * eps
            fd = (up - loss(q)) / (2 * eps)
            assert abs(fd - g.reshape(-1)[idx]) <= 2e-7 * scale + 1e-9, (name, idx, fd, g.reshape(-1)[idx])


def test_softmax_gate_is_library_softmax(o64):
    p = problem(9, T=20)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=9, mode=ob.MODE_TCR,
                     softmax_gate=True)
    rt = fw.route
    want = torch.softmax(torch_affinity(torch.from_numpy(p["X"]), torch.from_numpy(p["R"]), 2), dim=1).numpy()
    rows = np.nonzero(rt.slot_token >= 0)[0]
    assert len(rows) > 0 and rt.dropped > 0
    assert np.allclose(fw.gate[rows], want[rt.slot_token[rows], rows // rt.C_stride], rtol=1e-13, atol=0)
    assert np.all(fw.gate[rt.slot_token < 0] == 0)


def test_softmax_gate_dense_moe_fwd_bwd(o64):
    """Expert choice with C = T and the softmax gate is the general MoE form with
    G(x) = Softmax(affinities): forward and all five gradients against torch.autograd."""
    p = problem(10)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=12,
                     mode=ob.MODE_ECR, softmax_gate=True)
    bw = o64.backward(fw, p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], p["dY"])
    t = {k: torch.from_numpy(v).requires_grad_(k != "dY") for k, v in p.items()}
    gate = torch.softmax(torch_affinity(t["X"], t["R"], 2), dim=1)
    Y = 0
    for i in range(3):
        Y = Y + gate[:, i:i + 1] * torch_swiglu(t["X"], t["W1g"][i], t["W1u"][i], t["W2"][i])
    (Y * t["dY"]).sum().backward()
    assert np.allclose(fw.Y, Y.detach().numpy(), rtol=1e-12, atol=1e-13)
    for name, got in [("X", bw.dX), ("R", bw.dR), ("W1g", bw.dW1g), ("W1u", bw.dW1u), ("W2", bw.dW2)]:
        assert np.allclose(got, t[name].grad.numpy(), rtol=1e-10, atol=1e-12), name


def test_softmax_gate_gradients_by_finite_differences(o64):
    """Sparse selection (capacity active): the softmax still couples all experts of a token."""
    p = problem(11)
    kw = dict(D=2, k=2, capacity=5, mode=ob.MODE_TCR, softmax_gate=True)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], **kw)
    assert fw.route.dropped > 0
    bw = o64.backward(fw, p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], p["dY"])

    def loss(q):
        y = o64.forward(q["X"], q["R"], q["W1g"], q["W1u"], q["W2"], route=fw.route, **kw).Y
        return float((y * p["dY"]).sum())

    eps = 1e-6
    for name, g in dict(X=bw.dX, R=bw.dR).items():
        scale = np.abs(g).max()
        for idx in range(p[name].size):
            q = {k: v.copy() for k, v in p.items()}
            q[name].reshape(-1)[idx] += eps
            up = loss(q)
            q[name].reshape(-1)[idx] -= 2 * eps
            fd = (up - loss(q)) / (2 * eps)
            assert abs(fd - g.reshape(-1)[idx]) <= 2e-7 * scale + 1e-9, (name, idx, fd, g.reshape(-1)[idx])


def test_load_statistics(o64):
    p = problem(12, T=24)
    # expert choice with C = T: every expert processes every token; its mean gate is the column mean
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=24, mode=ob.MODE_ECR)
    load, gm = o64.load_stats(fw.route)
    assert np.array_equal(load, np.ones(3))
    assert np.allclose(gm, fw.delta.mean(axis=0), rtol=1e-13, atol=1e-15)
    # token choice under an active capacity: loads add up to the rows kept, and the summed gates are
    # what combining rows of ones gives
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=9, mode=ob.MODE_TCR)
    rt = fw.route
    load, gm = o64.load_stats(rt)
    assert rt.dropped > 0 and np.allclose(load * 24, rt.counts) and abs(load.sum() * 24 - rt.counts.sum()) < 1e-12
    ones = np.ones((3 * rt.C_stride, 1))
    assert abs(gm.sum() * 24 - o64.combine(ones, rt).sum()) < 1e-12
    by_hand = [sum(fw.delta[rt.slot_token[i * rt.C_stride + q], i] for q in range(rt.counts[i])) / 24 for i in range(3)]
    assert np.allclose(gm, by_hand, rtol=1e-13)


def test_router_gradient_orthogonality(o64):
    """The cosine ignores the scale of x_t and of R_i, so the router path's gradient
    satisfies <dX_router[t], x_t> = 0 and <dR_i, R_i> = 0."""
    p = problem(6)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=6, mode=ob.MODE_TCR)
    bw = o64.backward(fw, p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], p["dY"])
    dX_router = bw.dX - bw.dX_ffn
    assert np.abs(dX_router).max() > 1e-3
    assert np.allclose((dX_router * p["X"]).sum(1), 0, atol=1e-12)
    assert np.allclose((bw.dR * p["R"]).sum(1), 0, atol=1e-12)


def test_ffn_down_is_the_second_half_of_the_ffn(o64):
    p = problem(8)
    fw = o64.forward(p["X"], p["R"], p["W1g"], p["W1u"], p["W2"], D=2, k=2, capacity=6, mode=ob.MODE_TCR)
    assert np.array_equal(o64.expert_ffn_down(fw.H, fw.route, p["W2"]), fw.O)
    t = torch.from_numpy
    r = int(np.nonzero(fw.route.slot_token >= 0)[0][3])
    e = r // fw.route.C_stride
    assert np.allclose(fw.O[r], (t(p["W2"][e]) @ t(fw.H[r])).numpy(), rtol=1e-13, atol=1e-14)


def test_f32_layer_close_to_f64(o32, o64):
    w = gw.scaled(gw.WORKLOADS["tiny"], T=128, h=64)
    inp = gw.make_inputs(w)
    kw = dict(D=w.D, k=w.k, capacity=w.capacity, mode=ob.MODE_TCR)
    a = o32.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], **kw)
    b = o64.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], route=a.route, **kw)
    assert np.max(np.abs(a.Y - b.Y)) <= 1e-5 * np.sqrt((b.Y ** 2).mean())
    ga = o32.backward(a, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    gb = o64.backward(b, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    for f in ("dX", "dR", "dW1g", "dW1u", "dW2"):
        x, y = getattr(ga, f), getattr(gb, f)
        assert np.max(np.abs(x - y)) <= 2e-5 * np.sqrt((y ** 2).mean()), f


def test_oracle_is_thread_count_independent(o32):
    w = gw.scaled(gw.WORKLOADS["tiny"], T=96, h=32)
    inp = gw.make_inputs(w)
    kw = dict(D=w.D, k=w.k, capacity=w.capacity, mode=ob.MODE_TCR)
    n = ob.set_threads(0)
    try:
        ob.set_threads(1)
        a = o32.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], **kw)
        ga = o32.backward(a, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
        ob.set_threads(4)
        b = o32.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], **kw)
        gb = o32.backward(b, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    finally:
        ob.set_threads(n)
    assert np.array_equal(a.Y, b.Y)
    for f in ("dX", "dR", "dW1g", "dW1u", "dW2"):
        assert np.array_equal(getattr(ga, f), getattr(gb, f))


def test_storage_grid_composition_reduces_to_the_oracle_without_rounding(o32):
    """The stage-by-stage composition the GPU tests use as their sharp reference
    (harness.storage_grid_reference) rounds nothing for an fp32 layer, so it must reproduce the
    oracle's own forward and backward: same stages, same order, only split at the stored tensors
    (dXp as two products with the transposed weights, weight gradients expert by expert)."""
    from tests import harness as hz
    w = gw.scaled(gw.WORKLOADS["tiny"], T=160, h=48)
    inp = gw.make_inputs(w)
    for soft in (False, True):
        fw = o32.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k,
                         capacity=w.capacity, mode=ob.MODE_TCR, softmax_gate=soft)
        bw = o32.backward(fw, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
        g = hz.storage_grid_reference(o32, w, inp, fw, softmax_gate=soft)
        used = fw.route.slot_token >= 0
        for nm, ref in (("G", fw.G), ("U", fw.U), ("H", fw.H), ("O", fw.O), ("dO", bw.dO), ("dG", bw.dG),
                        ("dU", bw.dU), ("dXp", bw.dXp)):
            a, b = getattr(g, nm)[used], ref[used]
            assert np.max(np.abs(a - b)) <= 2e-6 * np.sqrt((b.astype(np.float64) ** 2).mean()), nm
        for nm, ref in (("Y", fw.Y), ("dX", bw.dX), ("dR", bw.dR), ("dW1g", bw.dW1g), ("dW1u", bw.dW1u),
                        ("dW2", bw.dW2), ("dgate", bw.dgate)):
            a = getattr(g, nm)
            assert np.max(np.abs(a - ref)) <= 2e-6 * np.sqrt((ref.astype(np.float64) ** 2).mean()), nm
    # and on a bf16 workload every stored tensor of the composition lies on the bf16 grid
    wb = gw.scaled(gw.WORKLOADS["small"], T=96, d=128, D=8, E=4, h=64)
    inp = gw.make_inputs(wb)
    fw = o32.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=wb.D, k=wb.k,
                     capacity=wb.capacity, mode=ob.MODE_TCR)
    g = hz.storage_grid_reference(o32, wb, inp, fw)
    for nm in ("G", "U", "H", "O", "Y", "dO", "dG", "dU", "dXp", "dX", "dW1g", "dW1u", "dW2"):
        a = getattr(g, nm)
        assert np.array_equal(a, gw.round_to_bf16(a)), nm
