"""ctypes access to the CPU oracle (test infrastructure; never used by the product path).

`build()` compiles oracle/etr_oracle_c.cpp with g++; `Oracle("f32"|"f64")` wraps the
exported functions with numpy arrays.  Only tests, the smoke check and the CPU-baseline
leg of the benchmark may import this module.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libetr_oracle.so")
_SRC = [os.path.join(_HERE, "etr_oracle_c.cpp"), os.path.join(_HERE, "etr_oracle.hpp")]

MODE_TCR, MODE_ECR = 1, 2


def build(force: bool = False) -> str:
    stale = force or not os.path.exists(_SO) or any(
        os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC)
    if stale:
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp",
                               "-o", _SO, _SRC[0]])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.etr_oracle_capacity_lower_bound.restype = ctypes.c_double
        _lib.etr_oracle_capacity_lower_bound.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_double]
        _lib.etr_oracle_capacity_bound.restype = ctypes.c_int
        _lib.etr_oracle_capacity_bound.argtypes = [ctypes.c_int] * 5 + [ctypes.c_double]
        _lib.etr_oracle_mode_for_step.restype = ctypes.c_int
        _lib.etr_oracle_mode_for_step.argtypes = [ctypes.c_longlong, ctypes.c_longlong]
        _lib.etr_oracle_set_threads.restype = ctypes.c_int
        _lib.etr_oracle_set_threads.argtypes = [ctypes.c_int]
    return _lib


def set_threads(n: int) -> int:
    return lib().etr_oracle_set_threads(int(n))


def capacity_lower_bound(d, E, delta_star) -> float:
    return lib().etr_oracle_capacity_lower_bound(int(d), int(E), float(delta_star))


def capacity_bound(d, E, capacity, c_floor, adaptive, delta_star) -> int:
    return lib().etr_oracle_capacity_bound(int(d), int(E), int(capacity), int(c_floor),
                                           int(bool(adaptive)), float(delta_star))


def mode_for_step(step, switch_step) -> int:
    return lib().etr_oracle_mode_for_step(int(step), int(switch_step))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


class Oracle:
    """The oracle in one scalar type.  Arrays are C-contiguous numpy arrays."""

    def __init__(self, scalar: str = "f32"):
        assert scalar in ("f32", "f64")
        self.suf = scalar
        self.np = np.float32 if scalar == "f32" else np.float64
        self.lib = lib()

    def _f(self, name):
        return getattr(self.lib, f"etr_oracle_{name}_{self.suf}")

    def arr(self, a):
        return np.ascontiguousarray(a, dtype=self.np)

    # -- forward stages ------------------------------------------------------------------
    def affinity(self, X, R, D):
        X, R = self.arr(X), self.arr(R)
        T, d = X.shape
        E, m = R.shape
        assert m * D == d
        delta = np.empty((T, E), self.np)
        xnorm = np.empty(T, self.np)
        rnorm = np.empty(E, self.np)
        dmax = np.empty(1, self.np)
        self._f("affinity")(T, d, D, E, _p(X), _p(R), _p(delta), _p(xnorm), _p(rnorm), _p(dmax))
        return delta, xnorm, rnorm, self.np(dmax[0])

    def select(self, delta, k, mode, C, C_stride):
        delta = self.arr(delta)
        T, E = delta.shape
        r = SimpleNamespace(
            topk_idx=np.empty((T, k), np.int32), counts=np.empty(E, np.int32),
            slot_token=np.empty(E * C_stride, np.int32), gate=np.empty(E * C_stride, self.np),
            tok_ptr=np.empty(T + 1, np.int32), tok_row=np.full(E * C_stride, -1, np.int32),
            C=int(C), C_stride=int(C_stride), mode=int(mode), E=E, T=T, k=k)
        dropped = np.zeros(1, np.int32)
        unrouted = np.zeros(1, np.int32)
        self._f("select")(T, E, k, int(mode), int(C), int(C_stride), _p(delta), _p(r.topk_idx),
                          _p(r.counts), _p(r.slot_token), _p(r.gate), _p(r.tok_ptr), _p(r.tok_row),
                          _p(dropped), _p(unrouted))
        r.dropped, r.unrouted = int(dropped[0]), int(unrouted[0])
        return r

    def select_thresholded(self, delta, k, mode, C, C_stride, threshold_mode, tau_expert=float("inf"),
                           tau_token=float("inf")):
        """select() with the cut by a running sum of affinities (bit 0: expert side, bit 1: token side)."""
        delta = self.arr(delta)
        T, E = delta.shape
        r = SimpleNamespace(
            topk_idx=np.empty((T, k), np.int32), counts=np.empty(E, np.int32),
            slot_token=np.empty(E * C_stride, np.int32), gate=np.empty(E * C_stride, self.np),
            tok_ptr=np.empty(T + 1, np.int32), tok_row=np.full(E * C_stride, -1, np.int32),
            C=int(C), C_stride=int(C_stride), mode=int(mode), E=E, T=T, k=k)
        dropped = np.zeros(1, np.int32)
        unrouted = np.zeros(1, np.int32)
        f = self._f("select_thresholded")
        f.argtypes = [ctypes.c_int] * 7 + [ctypes.c_double] * 2 + [ctypes.c_void_p] * 9
        f(T, E, k, int(mode), int(C), int(C_stride), int(threshold_mode), float(tau_expert), float(tau_token),
          _p(delta), _p(r.topk_idx), _p(r.counts), _p(r.slot_token), _p(r.gate), _p(r.tok_ptr), _p(r.tok_row),
          _p(dropped), _p(unrouted))
        r.dropped, r.unrouted = int(dropped[0]), int(unrouted[0])
        return r

    def dispatch(self, X, route):
        X = self.arr(X)
        d = X.shape[1]
        Xp = np.empty((route.E * route.C_stride, d), self.np)
        self._f("dispatch")(route.E, route.C_stride, d, _p(X), _p(route.slot_token), _p(Xp))
        return Xp

    def ffn_row(self, x, W1g_i, W1u_i, W2_i):
        x, W1g_i, W1u_i, W2_i = map(self.arr, (x, W1g_i, W1u_i, W2_i))
        h, d = W1g_i.shape
        g, u, hh = (np.empty(h, self.np) for _ in range(3))
        o = np.empty(d, self.np)
        self._f("ffn_row")(d, h, _p(x), _p(W1g_i), _p(W1u_i), _p(W2_i), _p(g), _p(u), _p(hh), _p(o))
        return g, u, hh, o

    def expert_ffn(self, Xp, route, W1g, W1u, W2):
        Xp, W1g, W1u, W2 = map(self.arr, (Xp, W1g, W1u, W2))
        E, h, d = W1g.shape
        rows = E * route.C_stride
        G, U, H = (np.empty((rows, h), self.np) for _ in range(3))
        O = np.empty((rows, d), self.np)
        self._f("expert_ffn")(E, route.C_stride, d, h, _p(route.counts), _p(Xp), _p(W1g), _p(W1u),
                              _p(W2), _p(G), _p(U), _p(H), _p(O))
        return G, U, H, O

    def expert_ffn_down(self, H, route, W2):
        """O = H W2_i^T alone (the second half of the FFN on a given hidden activation)."""
        H, W2 = self.arr(H), self.arr(W2)
        E, d, h = W2.shape
        O = np.empty((E * route.C_stride, d), self.np)
        self._f("expert_ffn_down")(E, route.C_stride, d, h, _p(route.counts), _p(H), _p(W2), _p(O))
        return O

    def combine(self, O, route, gate=None):
        O = self.arr(O)
        gate = self.arr(route.gate if gate is None else gate)
        d = O.shape[1]
        Y = np.empty((route.T, d), self.np)
        self._f("combine")(route.T, d, _p(route.tok_ptr), _p(route.tok_row), _p(gate), _p(O), _p(Y))
        return Y

    # -- backward stages -----------------------------------------------------------------
    def combine_bwd(self, dY, O, route, gate=None):
        dY, O = self.arr(dY), self.arr(O)
        gate = self.arr(route.gate if gate is None else gate)
        d = O.shape[1]
        dO = np.empty_like(O)
        dgate = np.empty(O.shape[0], self.np)
        self._f("combine_bwd")(route.E, route.C_stride, d, _p(route.slot_token), _p(gate), _p(dY),
                               _p(O), _p(dO), _p(dgate))
        return dO, dgate

    def ffn_row_bwd(self, go, g, u, W1g_i, W1u_i, W2_i):
        go, g, u, W1g_i, W1u_i, W2_i = map(self.arr, (go, g, u, W1g_i, W1u_i, W2_i))
        h, d = W1g_i.shape
        dg, du = np.empty(h, self.np), np.empty(h, self.np)
        dxp = np.empty(d, self.np)
        self._f("ffn_row_bwd")(d, h, _p(go), _p(g), _p(u), _p(W1g_i), _p(W1u_i), _p(W2_i),
                               _p(dg), _p(du), _p(dxp))
        return dg, du, dxp

    def ffn_weight_grads(self, dOe, He, dGe, dUe, Xpe):
        dOe, He, dGe, dUe, Xpe = map(self.arr, (dOe, He, dGe, dUe, Xpe))
        n, d = dOe.shape
        h = He.shape[1]
        dW1g, dW1u = np.empty((h, d), self.np), np.empty((h, d), self.np)
        dW2 = np.empty((d, h), self.np)
        self._f("ffn_weight_grads")(n, d, h, _p(dOe), _p(He), _p(dGe), _p(dUe), _p(Xpe),
                                    _p(dW1g), _p(dW1u), _p(dW2))
        return dW1g, dW1u, dW2

    def expert_ffn_bwd(self, dO, Xp, G, U, H, route, W1g, W1u, W2):
        dO, Xp, G, U, H, W1g, W1u, W2 = map(self.arr, (dO, Xp, G, U, H, W1g, W1u, W2))
        E, h, d = W1g.shape
        dG, dU = np.empty_like(G), np.empty_like(U)
        dXp = np.empty_like(Xp)
        dW1g, dW1u, dW2 = np.empty_like(W1g), np.empty_like(W1u), np.empty_like(W2)
        self._f("expert_ffn_bwd")(E, route.C_stride, d, h, _p(route.counts), _p(dO), _p(Xp), _p(G),
                                  _p(U), _p(H), _p(W1g), _p(W1u), _p(W2), _p(dG), _p(dU), _p(dXp),
                                  _p(dW1g), _p(dW1u), _p(dW2))
        return dG, dU, dXp, dW1g, dW1u, dW2

    def dispatch_bwd(self, dXp, route):
        dXp = self.arr(dXp)
        d = dXp.shape[1]
        dX = np.empty((route.T, d), self.np)
        self._f("dispatch_bwd")(route.T, d, _p(route.tok_ptr), _p(route.tok_row), _p(dXp), _p(dX))
        return dX

    def select_bwd(self, dgate, route):
        dgate = self.arr(dgate)
        dd = np.empty((route.T, route.E), self.np)
        self._f("select_bwd")(route.T, route.E, route.C_stride, _p(route.slot_token), _p(dgate), _p(dd))
        return dd

    def softmax_gate(self, delta, route):
        """Gates of the softmax variant: softmax of each token's affinities over all experts."""
        delta = self.arr(delta)
        gate = np.empty(route.E * route.C_stride, self.np)
        self._f("softmax_gate")(route.T, route.E, route.C_stride, _p(delta), _p(route.slot_token), _p(gate))
        return gate

    def softmax_gate_bwd(self, delta, dgate, route):
        delta, dgate = self.arr(delta), self.arr(dgate)
        dd = np.empty((route.T, route.E), self.np)
        self._f("softmax_gate_bwd")(route.T, route.E, route.C_stride, _p(delta), _p(route.slot_token),
                                    _p(dgate), _p(dd))
        return dd

    def load_stats(self, route, gate=None):
        """(load, gate_mean): tokens per expert / T, and summed gates per expert / T."""
        gate = self.arr(route.gate if gate is None else gate)
        load, gm = np.empty(route.E, self.np), np.empty(route.E, self.np)
        self._f("load_stats")(route.T, route.E, route.C_stride, _p(route.counts), _p(route.slot_token),
                              _p(gate), _p(load), _p(gm))
        return load, gm

    def affinity_bwd(self, X, R, D, delta, xnorm, rnorm, ddelta, dX):
        """Accumulates the router path's gradient into dX (in place); returns (dX, dR)."""
        X, R, delta, xnorm, rnorm, ddelta = map(self.arr, (X, R, delta, xnorm, rnorm, ddelta))
        assert dX.dtype == self.np and dX.flags.c_contiguous
        T, d = X.shape
        E, m = R.shape
        dR = np.empty((E, m), self.np)
        self._f("affinity_bwd")(T, d, D, E, _p(X), _p(R), _p(delta), _p(xnorm), _p(rnorm),
                                _p(ddelta), _p(dX), _p(dR))
        return dX, dR

    # -- the whole layer: the stages above in order ---------------------------------------
    def forward(self, X, R, W1g, W1u, W2, *, D, k, capacity, C_stride=None, mode=None, step=0,
                switch_step=0, adaptive=False, c_floor=1, delta_max_override=-1.0, route=None,
                softmax_gate=False, threshold_mode=0, tau_expert=float("inf"), tau_token=float("inf")):
        d = X.shape[1]
        E = R.shape[0]
        if C_stride is None:
            C_stride = (capacity + 127) // 128 * 128
        delta, xnorm, rnorm, dmax = self.affinity(X, R, D)
        if route is None:
            if mode is None:
                mode = mode_for_step(step, switch_step)
            dstar = float(dmax) if delta_max_override < 0 else float(delta_max_override)
            C = capacity_bound(d, E, capacity, c_floor, adaptive, dstar)
            if threshold_mode:
                route = self.select_thresholded(delta, k, mode, C, C_stride, threshold_mode, tau_expert, tau_token)
            else:
                route = self.select(delta, k, mode, C, C_stride)
            gate = route.gate
        else:  # frozen selection: gates re-read from this call's affinities
            gate = np.zeros(E * route.C_stride, self.np)
            v = route.slot_token >= 0
            rows = np.nonzero(v)[0]
            gate[rows] = delta[route.slot_token[rows], rows // route.C_stride]
        if softmax_gate:
            gate = self.softmax_gate(delta, route)
        Xp = self.dispatch(X, route)
        G, U, H, O = self.expert_ffn(Xp, route, W1g, W1u, W2)
        Y = self.combine(O, route, gate)
        return SimpleNamespace(delta=delta, xnorm=xnorm, rnorm=rnorm, delta_max=dmax, route=route,
                               gate=gate, Xp=Xp, G=G, U=U, H=H, O=O, Y=Y, D=D, softmax_gate=softmax_gate)

    def backward(self, fwd, X, R, W1g, W1u, W2, dY):
        rt = fwd.route
        dO, dgate = self.combine_bwd(dY, fwd.O, rt, fwd.gate)
        dG, dU, dXp, dW1g, dW1u, dW2 = self.expert_ffn_bwd(dO, fwd.Xp, fwd.G, fwd.U, fwd.H, rt,
                                                            W1g, W1u, W2)
        dX_ffn = self.dispatch_bwd(dXp, rt)
        if getattr(fwd, "softmax_gate", False):
            ddelta = self.softmax_gate_bwd(fwd.delta, dgate, rt)
        else:
            ddelta = self.select_bwd(dgate, rt)
        dX = dX_ffn.copy()
        dX, dR = self.affinity_bwd(X, R, fwd.D, fwd.delta, fwd.xnorm, fwd.rnorm, ddelta, dX)
        return SimpleNamespace(dO=dO, dgate=dgate, dG=dG, dU=dU, dXp=dXp, dW1g=dW1g, dW1u=dW1u,
                               dW2=dW2, dX_ffn=dX_ffn, ddelta=ddelta, dX=dX, dR=dR)
