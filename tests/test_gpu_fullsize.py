"""Parity at the full sizes of the five workloads (and of the Mixtral-shaped Top-1 workload), in the launch configuration the benchmark
times (etr_layer_forward + etr_layer_backward, default GEMM path).

The routing half is compared in full: the oracle computes every affinity and the complete
selection on the CPU, and every map must match (bit-exact outside the 1e-5 score margin).
The FFN half is too large for the CPU in full (up to 20 TFLOP), so it is compared on
samples the oracle computes one by one:
  * one whole expert: every row of G, U, H, O, dG, dU, dXp and its slices dW1g[i], dW1u[i],
    dW2[i], dR[i];
  * sampled tokens (several rows in different experts, and unrouted tokens): Y[t], dX[t];
  * sampled hidden units of other experts: exact slices dW1g[i][B,:], dW1u[i][B,:], dW2[i][:,B];
and on properties that hold at any size (pad rows zero, unrouted tokens get zeros).
"""
import os
from types import SimpleNamespace

import numpy as np
import pytest
import torch

from gen import workloads as gw
from oracle import binding as ob
from tests import harness as hz

pytestmark = pytest.mark.gpu
etr = hz.etr

# workload, delta_max given to both sides (None: the measured one), rows of the chosen expert that are
# checked (None: all of them, and with them the expert's whole weight gradients)
FULL = {
    "small": (gw.WORKLOADS["small"], -1.0, None),
    "mid": (gw.WORKLOADS["mid"], -1.0, None),
    # the adaptive-switch sweep: all eight steps with the supplied delta_max schedule (C walks from 1280 down
    # to 769, five steps in token choice and three in expert choice), and the first with the measured one
    **{f"sweep_step{gw.SWEEP_STEPS[i]}": (gw.sweep_point(i), gw.SWEEP_DELTA_MAX[i], None) for i in range(8)},
    "sweep_step0_measured": (gw.sweep_point(0), None, None),
    "large": (gw.WORKLOADS["large"], None, None),
    "mixtral_top1": (gw.WORKLOADS["mixtral_top1"], None, 24),     # 1 GFLOP per row on the CPU
}
if os.environ.get("ETR_SKIP_LARGE"):
    FULL.pop("large")
    FULL.pop("mixtral_top1")


# C = ceil(exp(d dm^2 / (2 - dm^2)) / E) for d = 2048, E = 32 at the eight supplied values of delta_max
SWEEP_C = (1280, 1234, 1151, 1088, 1025, 897, 831, 769)


def sub_route(E, Cs, n, T):
    """Route of a single expert holding rows 0..n-1 (tokens 0..n-1), for sub-problems."""
    st = np.full(Cs, -1, np.int32)
    st[:n] = np.arange(n, dtype=np.int32)
    return SimpleNamespace(E=1, C_stride=Cs, T=T, counts=np.array([n], np.int32), slot_token=st,
                           tok_ptr=np.arange(T + 1, dtype=np.int32).clip(max=n),
                           tok_row=np.arange(Cs, dtype=np.int32))


@pytest.mark.parametrize("name", list(FULL))
def test_full_size(name):
    w, dm, expert_rows = FULL[name]
    mode = hz.mode_of(w)
    o = ob.Oracle("f32")
    inp = gw.make_inputs(w)
    X, R, dY = inp["X"], inp["R"], inp["dY"]
    W1g, W1u, W2 = inp["W1g"], inp["W1u"], inp["W2"]
    T, d, E, h, D, Cs = w.T, w.d, w.E, w.h, w.D, w.C_stride
    tol = 2e-2

    # ---- oracle routing, in full -----------------------------------------------------------------
    delta, xnorm, rnorm, dmax = o.affinity(X, R, D)
    override = float(dmax) if dm is None else dm      # capacity parity: both sides clamp the same C
    C = ob.capacity_bound(d, E, w.capacity, 1, w.adaptive, override)
    ref = o.select(delta, w.k, mode, C, Cs)
    if name.startswith("sweep_step") and dm is not None:      # the schedule walks C through the interior of its clamp
        assert C == SWEEP_C[gw.SWEEP_DELTA_MAX.index(dm)]

    # ---- device: the timed path (measured delta_max) and the parity path (oracle's delta_max) -----
    dev = hz.upload(w, inp)
    out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
               dW1g=torch.empty_like(dev.W1g), dW1u=torch.empty_like(dev.W1u), dW2=torch.empty_like(dev.W2))
    if dm is None and w.adaptive:
        cfg_m = hz.make_cfg(w)
        buf_m = etr.LayerBuffers(cfg_m)
        etr.layer_forward(cfg_m, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf_m, out["Y"])
        st_m = buf_m.read_stats()
        assert abs(st_m.delta_max - float(dmax)) <= 1e-5 * abs(float(dmax))
        c_m = ob.capacity_bound(d, E, w.capacity, 1, True, st_m.delta_max)
        assert st_m.C == c_m and abs(st_m.C - C) <= 1
        del buf_m
    cfg = hz.make_cfg(w, delta_max_override=override if w.adaptive else -1.0)
    buf = etr.LayerBuffers(cfg)
    for t in (buf.Xp, buf.G, buf.U, buf.H, buf.O, buf.dO, buf.dG, buf.dU, buf.dXp):
        t.fill_(float("nan"))
    etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
    etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                       out["dW1g"], out["dW1u"], out["dW2"])
    torch.cuda.synchronize()
    st = buf.read_stats()
    assert st.error_word == 0
    got = hz.route_from_buffers(buf, cfg)
    delta_dev = hz.to_np(buf.delta)
    hz.assert_affinity_close(delta_dev, delta)
    assert np.allclose(hz.to_np(buf.xnorm), xnorm, rtol=2e-6)
    hz.check_route_structure(delta_dev, got, mode)
    hz.assert_routes_match(delta, ref, got, mode)
    counts = got.counts
    padded = (np.arange(Cs)[None, :] < ((counts + 127) // 128 * 128)[:, None]).reshape(-1)
    used = (np.arange(Cs)[None, :] < counts[:, None]).reshape(-1)

    # ---- properties at any size ---------------------------------------------------------------------
    pad_rows = torch.from_numpy(np.nonzero(padded & ~used)[0]).cuda()
    for nm in ("Xp", "G", "U", "H", "O", "dO", "dG", "dU", "dXp"):
        t = getattr(buf, nm)
        assert bool((t[pad_rows] == 0).all()), f"{nm}: pad rows must be zero"
    unrouted = torch.from_numpy(np.nonzero(np.diff(got.tok_ptr) == 0)[0]).cuda()
    assert bool((out["Y"][unrouted] == 0).all()) and bool((out["dX"][unrouted] == 0).all())
    sl = torch.from_numpy(got.slot_token[used].astype(np.int64)).cuda()
    assert torch.equal(buf.Xp[torch.from_numpy(np.nonzero(used)[0]).cuda()], dev.X[sl])

    # ---- one whole expert -------------------------------------------------------------------------------
    ragged = [i for i in range(E) if counts[i] % 128 != 0 and counts[i] > 0]
    i = ragged[len(ragged) // 2] if ragged else E - 1
    n_all = int(counts[i])
    n = n_all if expert_rows is None else min(n_all, expert_rows)      # rows are independent of each other
    r0 = i * Cs
    toks = got.slot_token[r0:r0 + n]
    gate = got.gate[r0:r0 + n]
    Cs1 = (n + 127) // 128 * 128
    rt1 = sub_route(1, Cs1, n, n)
    Xe = np.zeros((Cs1, d), np.float32)
    Xe[:n] = X[toks]
    G, U, H, O = o.expert_ffn(Xe, rt1, W1g[i:i + 1], W1u[i:i + 1], W2[i:i + 1])
    rows = slice(r0, r0 + n)
    hz.assert_close_rms(hz.to_np(buf.G[rows]), G[:n], tol, "G")
    hz.assert_close_rms(hz.to_np(buf.U[rows]), U[:n], tol, "U")
    hz.assert_close_rms(hz.to_np(buf.H[rows]), H[:n], tol, "H")
    hz.assert_close_rms(hz.to_np(buf.O[rows]), O[:n], tol, "O", chain=2)
    dO = np.zeros((Cs1, d), np.float32)
    dO[:n] = gate[:, None] * dY[toks]
    dgate = (dY[toks].astype(np.float64) * O[:n]).sum(1)
    hz.assert_close_rms(hz.to_np(buf.dO[rows]), dO[:n], tol, "dO")
    hz.assert_close_rms(hz.to_np(buf.dgate[rows]), dgate, tol, "dgate", chain=2)
    dG, dU, dXp, dW1g_i, dW1u_i, dW2_i = o.expert_ffn_bwd(dO, Xe, G, U, H, rt1, W1g[i:i + 1],
                                                           W1u[i:i + 1], W2[i:i + 1])
    hz.assert_close_rms(hz.to_np(buf.dG[rows]), dG[:n], tol, "dG", chain=3)
    hz.assert_close_rms(hz.to_np(buf.dU[rows]), dU[:n], tol, "dU", chain=3)
    hz.assert_close_rms(hz.to_np(buf.dXp[rows]), dXp[:n], tol, "dXp", chain=5)
    if n == n_all:          # sums over all the expert's rows
        frac = hz.dw1_outlier_fraction(w)
        hz.assert_close_rms(hz.to_np(out["dW1g"][i]), dW1g_i[0], tol, "dW1g[i]", chain=6, outlier_fraction=frac)
        hz.assert_close_rms(hz.to_np(out["dW1u"][i]), dW1u_i[0], tol, "dW1u[i]", chain=6, outlier_fraction=frac)
        hz.assert_close_rms(hz.to_np(out["dW2"][i]), dW2_i[0], tol, "dW2[i]", chain=4)
        # dR[i] from this expert's tokens only
        dd = np.zeros((n, E), np.float32)
        dd[:, i] = dgate
        _, dR_sub = o.affinity_bwd(X[toks], R, D, delta[toks], xnorm[toks], rnorm, dd, np.zeros((n, d), np.float32))
        hz.assert_close_rms(hz.to_np(out["dR"][i]), dR_sub[i], tol, "dR[i]", chain=4)

    # ---- sampled tokens: Y[t] and dX[t] through every row of the token ------------------------------------------
    rng = np.random.default_rng(w.seed)
    nrows_t = np.diff(got.tok_ptr)
    routed = np.nonzero(nrows_t > 0)[0]
    multi = np.nonzero(nrows_t > 1)[0]
    n_tok = 6 if expert_rows is None else 3
    pick = list(rng.choice(routed, n_tok, replace=False)) + (list(rng.choice(multi, min(4, len(multi)), replace=False)) if len(multi) else [])
    y_ref, dx_ref = np.zeros((len(pick), d)), np.zeros((len(pick), d), np.float32)
    for j, t in enumerate(pick):
        dx = np.zeros(d, np.float64)
        dd = np.zeros((1, E), np.float32)
        for q in range(got.tok_ptr[t], got.tok_ptr[t + 1]):
            r = int(got.tok_row[q])
            e = r // Cs
            g, u, hh, oo = o.ffn_row(X[t], W1g[e], W1u[e], W2[e])
            y_ref[j] += float(got.gate[r]) * oo.astype(np.float64)
            dd[0, e] = float((dY[t].astype(np.float64) * oo).sum())
            _, _, dxp = o.ffn_row_bwd(got.gate[r] * dY[t], g, u, W1g[e], W1u[e], W2[e])
            dx += dxp
        dx32 = dx.astype(np.float32)[None, :].copy()
        o.affinity_bwd(X[t:t + 1], R, D, delta[t:t + 1], xnorm[t:t + 1], rnorm, dd, dx32)
        dx_ref[j] = dx32[0]
    idx = torch.from_numpy(np.asarray(pick, dtype=np.int64)).cuda()
    # the scale of each comparison is the RMS of the oracle's own rows (all sampled tokens are routed)
    hz.assert_close_rms(hz.to_np(out["Y"][idx]), y_ref, tol, "Y[sampled tokens]", chain=4)
    hz.assert_close_rms(hz.to_np(out["dX"][idx]), dx_ref, tol, "dX[sampled tokens]", chain=6)

    # ---- sampled hidden units of two other experts: exact slices of the weight gradients ----------------------
    others = [e for e in rng.permutation(E) if e != i and counts[e] > 0][:2]
    for e in others:
        n = int(counts[e])
        r0 = e * Cs
        toks = got.slot_token[r0:r0 + n]
        Cs1 = (n + 127) // 128 * 128
        rt1 = sub_route(1, Cs1, n, n)
        Xe = np.zeros((Cs1, d), np.float32)
        Xe[:n] = X[toks]
        dO = np.zeros((Cs1, d), np.float32)
        dO[:n] = got.gate[r0:r0 + n, None] * dY[toks]
        B = np.sort(rng.choice(h, 8, replace=False))
        w1g, w1u, w2 = W1g[e][B][None], W1u[e][B][None], np.ascontiguousarray(W2[e][:, B])[None]
        G, U, H, _ = o.expert_ffn(Xe, rt1, w1g, w1u, w2)
        _, _, _, s_dW1g, s_dW1u, s_dW2 = o.expert_ffn_bwd(dO, Xe, G, U, H, rt1, w1g, w1u, w2)
        for nm, ref_slice, chain, take in (("dW1g", s_dW1g[0], 6, lambda a: a[B]),
                                           ("dW1u", s_dW1u[0], 6, lambda a: a[B]),
                                           ("dW2", s_dW2[0], 4, lambda a: a[:, B])):
            hz.assert_close_rms(take(hz.to_np(out[nm][e])), ref_slice, tol, f"{nm}[{e}] slice", chain=chain)
