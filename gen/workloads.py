"""Seeded synthetic inputs for the ETR MoE layer.

This module only draws random tensors; it contains none of the layer's
arithmetic.  Both the CPU oracle's tests and the CUDA path's tests/bench import
it, so the two sides see identical bits.

The paper trains Mixtral-style MoE blocks on a private corpus; neither the corpus
nor the weights exist here.  The inputs below reproduce the *structure* the paper
describes: token features that are isotropic and mutually near-orthogonal early in
training and block-clustered (within-cluster correlation > 0.8) late in training
(appendix "Token Feature Distribution"), and a skewed tokens-per-expert load
(the tokens-per-expert figure of the experiments section).

All tensors are returned as float32 numpy arrays whose values already lie on the
grid of the workload's storage dtype (for "bf16" workloads every value is exactly
representable in bfloat16), so converting them to that dtype is lossless.
"""
from __future__ import annotations

import math
import os
import zlib
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 0xE7120000


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    T: int            # tokens (batch x seq flattened; the paper's s)
    d: int            # hidden size
    D: int            # GrAP group size
    E: int            # experts (the paper's n)
    k: int            # experts per token (the paper's l)
    h: int            # FFN hidden size
    cf: float         # capacity factor
    dtype: str        # "f32" or "bf16": storage type of activations and weights
    mode: str         # "tcr" | "ecr" | "auto"
    adaptive: bool    # apply the adaptive capacity bound
    x_kind: str       # "iso" | "mix" | "skew"
    n_clusters: int = 0
    sigma: float = 0.5
    rho: float = 0.5
    step: int = 0
    switch_step: int = 1000
    ramp_steps: int = 2000

    @property
    def m(self) -> int:
        return self.d // self.D

    @property
    def capacity(self) -> int:
        return int(math.ceil(self.cf * self.T * self.k / self.E))

    @property
    def C_stride(self) -> int:
        return (self.capacity + 127) // 128 * 128

    @property
    def seed(self) -> int:
        return BASE_SEED + self.config_id


WORKLOADS = {
    "tiny": Workload("tiny", 1, T=512, d=256, D=4, E=8, k=2, h=512, cf=1.25, dtype="f32",
                     mode="tcr", adaptive=False, x_kind="iso", step=0),
    "small": Workload("small", 2, T=4096, d=1024, D=8, E=16, k=2, h=2816, cf=1.25, dtype="bf16",
                      mode="tcr", adaptive=False, x_kind="iso", step=10),
    "mid": Workload("mid", 3, T=16384, d=2048, D=8, E=32, k=2, h=1408, cf=1.0, dtype="bf16",
                    mode="ecr", adaptive=False, x_kind="mix", n_clusters=32, step=5000),
    "sweep": Workload("sweep", 4, T=16384, d=2048, D=16, E=32, k=2, h=1408, cf=1.25, dtype="bf16",
                      mode="auto", adaptive=True, x_kind="skew", n_clusters=32, step=0),
    "large": Workload("large", 5, T=65536, d=4096, D=16, E=64, k=2, h=2048, cf=1.0, dtype="bf16",
                      mode="ecr", adaptive=True, x_kind="mix", n_clusters=64, step=5000),
    # The expert shape of the paper's own model (Mixtral 8x7B: 8 experts, d=4096, h=14336) at its
    # sequence length, with Top-1 routing as in its efficiency runs; early training (TCR).
    "mixtral_top1": Workload("mixtral_top1", 6, T=32768, d=4096, D=16, E=8, k=1, h=14336, cf=1.0,
                             dtype="bf16", mode="tcr", adaptive=True, x_kind="mix", n_clusters=64, step=10),
}

# Training steps of the adaptive-switch sweep (five before the switch, three after)
SWEEP_STEPS = (0, 300, 600, 900, 999, 1000, 1500, 2000)
# A supplied delta_max schedule that walks the adaptive bound through the interior
# of its clamp for d=2048, E=32 (the measured batch maximum clamps to `capacity`).
SWEEP_DELTA_MAX = (0.10158, 0.10140, 0.10107, 0.10080, 0.10051, 0.09987, 0.09950, 0.09912)


def sweep_point(i: int) -> Workload:
    return replace(WORKLOADS["sweep"], name=f"sweep{i}", step=SWEEP_STEPS[i])


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some sizes replaced (used for small parity cases)."""
    return replace(w, **kw)


def _rng(w: Workload, tensor: str) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(
        np.random.SeedSequence([w.seed, zlib.crc32(tensor.encode())])))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even), kept as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


def _to_grid(w: Workload, a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if w.dtype == "bf16" else a


_CHUNK = 1 << 22


def _normal(w: Workload, tensor: str, shape, scale=1.0) -> np.ndarray:
    """N(0, scale^2) float32.  The tensor is cut into fixed chunks, each with its own
    counter-seeded stream, so the bits do not depend on how many threads fill it."""
    out = np.empty(shape, dtype=np.float32)
    flat = out.reshape(-1)
    tag = zlib.crc32(tensor.encode())
    sc = np.float32(scale)

    def fill(c):
        s = c * _CHUNK
        e = min(flat.size, s + _CHUNK)
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([w.seed, tag, c])))
        rng.standard_normal(e - s, dtype=np.float32, out=flat[s:e])
        if scale != 1.0:
            flat[s:e] *= sc

    n_chunks = (flat.size + _CHUNK - 1) // _CHUNK
    if n_chunks <= 1:
        for c in range(n_chunks):
            fill(c)
    else:
        with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, range(n_chunks)))
    return out


def expert_embeddings(w: Workload) -> np.ndarray:
    """R[E, m] fp32 with orthonormal rows: thin QR of an m x E Gaussian, R = Q^T,
    signs fixed so the triangular factor has a positive diagonal."""
    assert w.E <= w.m, "orthonormal rows need E <= d/D"
    g = _rng(w, "R").standard_normal((w.m, w.E))
    q, r = np.linalg.qr(g)
    q = q * np.sign(np.diag(r))[None, :]
    return np.ascontiguousarray(q.T, dtype=np.float32)


def _unit_rows(a: np.ndarray) -> np.ndarray:
    return a / np.linalg.norm(a, axis=1, keepdims=True)


def cluster_means(w: Workload, R: np.ndarray | None = None) -> np.ndarray:
    """Unit-norm cluster means in R^d (float64)."""
    u = _unit_rows(_rng(w, "means").standard_normal((w.n_clusters, w.d)))
    if w.x_kind == "mix":
        return u
    # "skew": each mean leans toward one expert's GrAP direction
    if R is None:
        R = expert_embeddings(w)
    lean = np.repeat(R.astype(np.float64), w.D, axis=1) / math.sqrt(w.D)     # unit rows in R^d
    idx = np.arange(w.n_clusters) % w.E
    mu = w.rho * lean[idx] + math.sqrt(1.0 - w.rho ** 2) * u
    return _unit_rows(mu)


def cluster_ids(w: Workload) -> np.ndarray:
    rng = _rng(w, "cluster_ids")
    if w.x_kind == "skew":
        p = (np.arange(w.n_clusters) + 1.0) ** -1.2
        p /= p.sum()
        return rng.choice(w.n_clusters, size=w.T, p=p).astype(np.int64)
    return rng.integers(0, w.n_clusters, size=w.T, dtype=np.int64)


def tokens(w: Workload, R: np.ndarray | None = None) -> np.ndarray:
    """X[T, d] on the workload's dtype grid."""
    eps = _normal(w, "X", (w.T, w.d))
    if w.x_kind == "iso":
        return _to_grid(w, eps)
    mu = cluster_means(w, R).astype(np.float32)
    cid = cluster_ids(w)
    noise = w.sigma / math.sqrt(w.d)
    if w.x_kind == "mix":
        x = eps
        x *= np.float32(noise)
        for s in range(0, w.T, 4096):
            x[s:s + 4096] += mu[cid[s:s + 4096]]
        return _to_grid(w, x)
    # "skew": isotropic at step 0, clustered at ramp_steps
    alpha = min(1.0, w.step / float(w.ramp_steps))
    x = eps
    x *= np.float32((1.0 - alpha) + alpha * noise)
    if alpha > 0.0:
        for s in range(0, w.T, 4096):
            x[s:s + 4096] += np.float32(alpha) * mu[cid[s:s + 4096]]
    return _to_grid(w, x)


def expert_weights(w: Workload):
    """W1g[E,h,d], W1u[E,h,d], W2[E,d,h] ~ N(0, 1/d) on the dtype grid."""
    std = 1.0 / math.sqrt(w.d)
    W1g = _to_grid(w, _normal(w, "W1g", (w.E, w.h, w.d), std))
    W1u = _to_grid(w, _normal(w, "W1u", (w.E, w.h, w.d), std))
    W2 = _to_grid(w, _normal(w, "W2", (w.E, w.d, w.h), std))
    return W1g, W1u, W2


def output_grad(w: Workload) -> np.ndarray:
    """dY[T, d] ~ N(0, 1) on the dtype grid."""
    return _to_grid(w, _normal(w, "dY", (w.T, w.d)))


def make_inputs(w: Workload, weights: bool = True) -> dict:
    R = expert_embeddings(w)
    out = {"R": R, "X": tokens(w, R), "dY": output_grad(w)}
    if weights:
        out["W1g"], out["W1u"], out["W2"] = expert_weights(w)
    return out
