"""Helpers shared by the GPU parity tests: upload seeded inputs, run the CUDA path through
the C ABI, and compare against the CPU oracle with the tolerances stated in the tests."""
from __future__ import annotations

from types import SimpleNamespace

import numpy as np
import torch

from gen import workloads as gw
from oracle import binding as ob
from paper_2406_00023_b200 import etr

MARGIN = 1e-5          # absolute affinity margin below which a routing decision is exempt


def mode_of(w: gw.Workload) -> int:
    if w.mode == "tcr":
        return ob.MODE_TCR
    if w.mode == "ecr":
        return ob.MODE_ECR
    return ob.mode_for_step(w.step, w.switch_step)


def make_cfg(w: gw.Workload, *, gemm_impl=etr.GEMM_AUTO, delta_max_override=-1.0, mode=None,
             fuse_dispatch=etr.FUSE_AUTO, gate_mode=etr.GATE_AFFINITY):
    m = mode_of(w) if mode is None else mode
    return etr.make_config(T=w.T, d=w.d, D=w.D, E=w.E, k=w.k, h=w.h, capacity=w.capacity,
                           dtype=etr.BF16 if w.dtype == "bf16" else etr.F32,
                           mode=etr.MODE_TCR if m == ob.MODE_TCR else etr.MODE_ECR,
                           step=w.step, switch_step=w.switch_step, adaptive=w.adaptive,
                           delta_max_override=delta_max_override, gemm_impl=gemm_impl,
                           fuse_dispatch=fuse_dispatch, gate_mode=gate_mode)


def to_dev(a: np.ndarray, w: gw.Workload | None = None, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is None and w is not None and a.dtype == np.float32:
        dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy() if t.dtype == torch.bfloat16 else t.detach().cpu().numpy()


def upload(w: gw.Workload, inp: dict) -> SimpleNamespace:
    d = SimpleNamespace()
    d.R = to_dev(inp["R"], dtype=torch.float32)
    for k in ("X", "dY", "W1g", "W1u", "W2"):
        if k in inp:
            setattr(d, k, to_dev(inp[k], w))
    return d


def route_from_buffers(buf: etr.LayerBuffers, cfg) -> SimpleNamespace:
    """Host copy of the device routing maps in the oracle's route format."""
    st = buf.read_stats()
    E, T, k = cfg.E, cfg.T, cfg.k
    Cs = etr.c_stride(cfg)
    r = SimpleNamespace(topk_idx=to_np(buf.topk_idx), counts=to_np(buf.counts),
                        slot_token=to_np(buf.slot_token), gate=to_np(buf.gate),
                        tok_ptr=to_np(buf.tok_ptr), tok_row=to_np(buf.tok_row).copy(),
                        C=st.C, C_stride=Cs, mode=st.mode, E=E, T=T, k=k,
                        dropped=st.dropped, unrouted=st.unrouted, rows_total=st.rows_total,
                        delta_max=st.delta_max)
    r.tok_row[r.rows_total:] = -1
    return r


def upload_route(buf: etr.LayerBuffers, rt) -> None:
    buf.topk_idx.copy_(torch.from_numpy(rt.topk_idx))
    buf.counts.copy_(torch.from_numpy(rt.counts))
    buf.slot_token.copy_(torch.from_numpy(rt.slot_token))
    buf.gate.copy_(torch.from_numpy(rt.gate.astype(np.float32)))
    buf.tok_ptr.copy_(torch.from_numpy(rt.tok_ptr))
    buf.tok_row.copy_(torch.from_numpy(rt.tok_row))


def assert_affinity_close(got, ref, what="delta"):
    """|got - ref| <= 1e-5 * max(|ref|, rms(ref)) element by element."""
    ref64 = ref.astype(np.float64)
    rms = np.sqrt((ref64 ** 2).mean())
    tol = 1e-5 * np.maximum(np.abs(ref64), rms)
    err = np.abs(got.astype(np.float64) - ref64)
    bad = err > tol
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside 1e-5 relative; worst {np.max(err / tol):.2f}x"


BF16_HALF_ULP = 2.0 ** -8     # worst-case relative error of rounding one value to bfloat16


def assert_close_rms(got, ref, rel, what, chain=1, rms=None):
    """|got - ref| <= rel * rms(ref) + chain * 2^-8 * |ref|, element by element.

    The first term is the target's bound (2e-2 of the reference tensor's RMS for bf16
    compute, 1e-4 for fp32).  The second exists only for bf16 storage (rel >= 1e-2) and
    covers what rounding to the bf16 grid does to a single large element, which no kernel
    writing bf16 can avoid: each rounding costs up to half an ulp, 2^-8 of the value (an
    element 5 RMS large already carries 2e-2 RMS of it).  `chain` is the number of
    bf16-stored tensors on the multiplicative path from the test's inputs to this output,
    the output's own store included: 1 for a stage fed with inputs already on the grid.

    For bf16 the bound is a max over millions of elements of an error whose RMS is a few
    tenths of a percent of rms(ref) per stored intermediate, i.e. it sits in the extreme
    tail; up to 2e-5 of the elements (at least one) may exceed it, none by more than 2x.
    fp32 comparisons allow no outliers."""
    storage = chain * BF16_HALF_ULP if rel >= 1e-2 else 0.0
    ref64 = ref.astype(np.float64)
    if rms is None:       # callers comparing a sample pass the RMS of the whole tensor
        rms = np.sqrt((ref64 ** 2).mean()) if ref.size else 0.0
    err = np.abs(got.astype(np.float64) - ref64)
    tol = rel * rms + storage * np.abs(ref64) + 1e-30
    ratio = err / tol
    n_bad = int((ratio > 1.0).sum())
    allowed = max(1, int(2e-5 * ref.size)) if rel >= 1e-2 else 0
    worst = float(ratio.max()) if ref.size else 0.0
    assert n_bad <= allowed and worst <= 2.0, (
        f"{what}: {n_bad} of {ref.size} elements outside tolerance (allowed {allowed}); worst "
        f"err {err.max():.3e}, rms {rms:.3e}, worst err/tol {worst:.2f}")
    return worst


def assert_routes_match(delta_ref: np.ndarray, ref, got, mode: int, margin: float = MARGIN):
    """Routing maps must be bit-identical wherever the oracle's score margin exceeds `margin`.

    Returns True if the two routes are identical everywhere.  Pairs (t, i) on which they
    differ must sit within `margin` of a decision boundary of the oracle: token t's k-th vs
    (k+1)-th affinity, or expert i's cut between its last kept and first dropped candidate.
    Whatever the differing pairs cannot influence must still be equal; the structure of the
    device maps is validated separately (check_route_structure)."""
    T, E = delta_ref.shape
    Cs = ref.C_stride
    assert got.C == ref.C, f"capacity {got.C} != {ref.C}"
    assert got.mode == ref.mode
    same = (np.array_equal(ref.counts, got.counts) and np.array_equal(ref.slot_token, got.slot_token)
            and np.array_equal(ref.tok_ptr, got.tok_ptr)
            and np.array_equal(ref.tok_row[:ref.tok_ptr[-1]], got.tok_row[:got.tok_ptr[-1]])
            and np.array_equal(ref.topk_idx, got.topk_idx))
    if same:
        return True
    k = ref.k
    srt = -np.sort(-delta_ref, axis=1)
    tok_margin = srt[:, k - 1] - srt[:, k] if (mode == ob.MODE_TCR and k < E) else np.full(T, np.inf)
    if mode == ob.MODE_TCR:
        diff_t = np.nonzero((ref.topk_idx != got.topk_idx).any(1))[0]
        assert np.all(tok_margin[diff_t] <= margin), "top-k differs outside the margin"
    for i in range(E):
        a = ref.slot_token[i * Cs:i * Cs + ref.counts[i]]
        b = got.slot_token[i * Cs:i * Cs + got.counts[i]]
        if np.array_equal(a, b):
            continue
        sym = np.setxor1d(a, b)
        cut = delta_ref[a, i].min() if len(a) else -np.inf
        near_cut = np.abs(delta_ref[sym, i] - cut) <= margin
        near_tok = tok_margin[sym] <= margin
        assert np.all(near_cut | near_tok), f"expert {i}: kept sets differ outside the margin"
        if not np.any(near_tok):
            assert len(a) == len(b)
    return False


def check_route_structure(delta_dev: np.ndarray, rt, mode: int):
    """Properties that hold for any valid route (used at sizes where maps are not compared
    slot by slot, and for margin-exempt differences): counts within C, ascending injective
    slots, gates equal to the device affinities bit for bit, CSR is the exact inverse."""
    T, E = delta_dev.shape
    Cs = rt.C_stride
    assert np.all(rt.counts >= 0) and np.all(rt.counts <= rt.C)
    sl = rt.slot_token.reshape(E, Cs)
    gt = rt.gate.reshape(E, Cs)
    pos = np.arange(Cs)[None, :]
    used = pos < rt.counts[:, None]
    assert np.all(sl[~used] == -1) and np.all(gt[~used] == 0)
    assert np.all(sl[used] >= 0) and np.all(sl[used] < T)
    asc = (np.diff(sl, axis=1) > 0) | ~used[:, 1:]
    assert np.all(asc)
    ei = np.broadcast_to(np.arange(E)[:, None], sl.shape)
    assert np.array_equal(gt[used], delta_dev[sl[used], ei[used]])
    if mode == ob.MODE_ECR:
        assert np.all(rt.counts == min(rt.C, T))
    # CSR inverse
    rows = np.nonzero(used.reshape(-1))[0]
    toks = rt.slot_token[rows]
    order = np.lexsort((rows, toks))
    assert rt.tok_ptr[0] == 0 and rt.tok_ptr[-1] == len(rows)
    assert np.array_equal(rt.tok_row[:len(rows)], rows[order])
    assert np.array_equal(np.diff(rt.tok_ptr), np.bincount(toks, minlength=T))
    assert rt.unrouted == int((np.diff(rt.tok_ptr) == 0).sum())
    n_cand = T * rt.k if mode == ob.MODE_TCR else T * E
    assert rt.dropped == n_cand - len(rows)
