"""Pins for the oracle's routing half: affinity, capacity, selection.

Each test checks the oracle against something the paper or the mathematics fixes
independently of the oracle's own code: the paper's closed-form W_aff, textbook
cosine through numpy, orthogonality, Bessel's inequality, invariances, hand-worked
C_min values, algebraic inversions of C_min, brute-force subset search, and the
set-level invariants of token choice and expert choice.
"""
import itertools
import math
import os

import numpy as np
import pytest

from gen import workloads as gw
from oracle import binding as ob

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def o32():
    return ob.Oracle("f32")


@pytest.fixture(scope="module")
def o64():
    return ob.Oracle("f64")


def rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ---------------------------------------------------------------- affinity ------------
def test_affinity_paper_closed_form(o64):
    """With one expert per group and R = I the layer is the paper's own W_aff: row i is
    n/d on segment i, so delta_ti = (sum of x_t over segment i) / (sqrt(d/n) ||x_t||)."""
    T, n, seg = 7, 6, 5
    d = n * seg
    X = rand((T, d), 1)
    delta, xnorm, rnorm, dmax = o64.affinity(X, np.eye(n), D=seg)
    W = np.zeros((n, d))
    for i in range(n):
        W[i, i * seg:(i + 1) * seg] = n / d
    ref = (X @ W.T) / (np.linalg.norm(X, axis=1)[:, None] * np.linalg.norm(W, axis=1)[None, :])
    assert np.allclose(delta, ref, rtol=0, atol=1e-14)
    seg_sum = X.reshape(T, n, seg).sum(-1)
    assert np.allclose(delta, seg_sum / (math.sqrt(seg) * np.linalg.norm(X, axis=1)[:, None]), atol=1e-14)
    assert dmax == delta.max()
    assert np.allclose(xnorm, np.linalg.norm(X, axis=1), rtol=1e-15)
    assert np.allclose(rnorm, 1.0)


def test_affinity_D1_is_textbook_cosine(o64):
    T, d, E = 9, 12, 5
    X, R = rand((T, d), 2), rand((E, d), 3)
    delta, *_ = o64.affinity(X, R, D=1)
    ref = (X @ R.T) / np.outer(np.linalg.norm(X, axis=1), np.linalg.norm(R, axis=1))
    assert np.allclose(delta, ref, atol=1e-14)


def test_affinity_general_R_matches_dense_W(o64):
    """General R: delta is the cosine between x_t and the d-vector w_i that spreads
    R_i[j]/D over group j (so the router is x -> avgpool -> R)."""
    T, D, m, E = 6, 3, 8, 4
    d = D * m
    X, R = rand((T, d), 4), rand((E, m), 5)
    delta, *_ = o64.affinity(X, R, D=D)
    W = np.repeat(R, D, axis=1) / D
    ref = (X @ W.T) / np.outer(np.linalg.norm(X, axis=1), np.linalg.norm(W, axis=1))
    assert np.allclose(delta, ref, atol=1e-14)


def test_affinity_orthogonality(o64):
    """Orthonormal R and x = c * expand(R_i): delta_ti = 1 and delta_tj = 0 for j != i."""
    w = gw.WORKLOADS["tiny"]
    R = gw.expert_embeddings(w).astype(np.float64)
    q, _ = np.linalg.qr(R.T)              # re-orthonormalise in double
    R = q.T * np.sign((q.T * R).sum(1))[:, None]
    X = 3.7 * np.repeat(R, w.D, axis=1)
    delta, *_ = o64.affinity(X, R, D=w.D)
    assert np.allclose(delta, np.eye(w.E), atol=1e-12)


def test_affinity_bessel_and_range(o32):
    for name in ("tiny", "small"):
        w = gw.scaled(gw.WORKLOADS[name], T=256)
        R = gw.expert_embeddings(w)
        X = gw.tokens(w, R)
        delta, *_ = o32.affinity(X, R, D=w.D)
        assert np.all(np.abs(delta) <= 1.0 + 1e-6)
        assert np.all((delta.astype(np.float64) ** 2).sum(1) <= 1.0 + 1e-5)


def test_affinity_bessel_equality_case(o64):
    """x constant inside every group and pooled vector in span(R): sum_i delta^2 = 1."""
    D, m, E = 4, 6, 6
    q, _ = np.linalg.qr(rand((m, E), 6))
    R = q.T
    z = rand((3, E), 7) @ R
    X = np.repeat(z, D, axis=1)
    delta, *_ = o64.affinity(X, R, D=D)
    assert np.allclose((delta ** 2).sum(1), 1.0, atol=1e-12)


def test_affinity_invariances(o64):
    T, D, m, E = 5, 2, 6, 3
    X, R = rand((T, D * m), 8), rand((E, m), 9)
    base, *_ = o64.affinity(X, R, D=D)
    assert np.allclose(o64.affinity(2.5 * X, R, D=D)[0], base, atol=1e-14)
    assert np.allclose(o64.affinity(X, R * np.array([[0.3], [7.0], [1.9]]), D=D)[0], base, atol=1e-14)
    assert np.allclose(o64.affinity(-X, R, D=D)[0], -base, atol=1e-14)


def test_affinity_zero_norm_guard(o32):
    X = np.zeros((2, 8), np.float32)
    X[1] = 1.0
    delta, xnorm, *_ = o32.affinity(X, np.eye(4, dtype=np.float32), D=2)
    assert np.all(delta[0] == 0) and xnorm[0] == 0
    assert np.allclose(delta[1], 0.5)


def test_affinity_f32_close_to_f64(o32, o64):
    w = gw.scaled(gw.WORKLOADS["small"], T=128)
    R = gw.expert_embeddings(w)
    X = gw.tokens(w, R)
    a, *_ = o32.affinity(X, R, D=w.D)
    b, *_ = o64.affinity(X, R, D=w.D)
    assert np.max(np.abs(a - b)) <= 2e-7 * max(1.0, np.abs(b).max())


# ---------------------------------------------------------------- capacity ------------
def test_cmin_hand_values():
    rows = [ln.split("#")[0].split() for ln in open(os.path.join(GOLDEN, "cmin_hand_values.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for d, n, dm, want in rows:
        got = ob.capacity_lower_bound(int(d), int(n), float(dm))
        assert abs(got - float(want)) <= 1e-6 * float(want) + 5e-8 * 10 ** math.ceil(math.log10(float(want)))


def test_cmin_inversions():
    """Solving the closed form for delta: d x/(2-x) = L  <=>  x = 2L/(d+L).  L = ln n gives
    C_min = 1; L = ln(T n) gives C_min = T (the isotropic early-training case)."""
    assert ob.capacity_lower_bound(512, 16, 0.0) == pytest.approx(1 / 16, rel=1e-15)
    for d, n, T in [(256, 8, 512), (2048, 32, 16384), (4096, 64, 65536)]:
        L = math.log(n)
        assert ob.capacity_lower_bound(d, n, math.sqrt(2 * L / (d + L))) == pytest.approx(1.0, rel=1e-12)
        L = math.log(T * n)
        assert ob.capacity_lower_bound(d, n, math.sqrt(2 * L / (d + L))) == pytest.approx(T, rel=1e-11)
    # delta = 1: exponent is exactly d
    assert ob.capacity_lower_bound(8, 2, 1.0) == pytest.approx(math.e ** 8 / 2, rel=1e-14)


def test_capacity_bound_clamp_and_monotone():
    d, E, cap = 2048, 32, 1280
    assert ob.capacity_bound(d, E, cap, 1, 0, 0.5) == cap          # not adaptive
    assert ob.capacity_bound(d, E, cap, 1, 1, 0.0) == 1            # ceil(1/32) = 1
    assert ob.capacity_bound(d, E, cap, 64, 1, 0.0) == 64          # floor clamp
    assert ob.capacity_bound(d, E, cap, 1, 1, 1.0) == cap          # overflow clamps to capacity
    assert ob.capacity_bound(d, E, cap, 1, 1, 0.1) == 922          # ceil(921.24)
    prev = 0
    for dm in np.linspace(0, 0.2, 201):
        c = ob.capacity_bound(d, E, cap, 1, 1, float(dm))
        assert 1 <= c <= cap and c >= prev
        prev = c
    # the sweep schedule walks C down through the interior of the clamp (about 40 %)
    cs = [ob.capacity_bound(d, E, cap, 1, 1, dm) for dm in gw.SWEEP_DELTA_MAX]
    assert cs[0] == cap and all(a >= b for a, b in zip(cs, cs[1:])) and cs[-1] < 0.61 * cap
    assert ob.capacity_bound(d, E, cap, 1, 1, -0.3) == 1           # negative clamps to 0


def test_mode_switch():
    assert ob.mode_for_step(0, 1000) == ob.MODE_TCR
    assert ob.mode_for_step(999, 1000) == ob.MODE_TCR
    assert ob.mode_for_step(1000, 1000) == ob.MODE_ECR
    assert ob.mode_for_step(5000, 1000) == ob.MODE_ECR


# ---------------------------------------------------------------- selection -----------
def brute_token_side(row, k):
    best = None
    for sub in itertools.combinations(range(len(row)), k):
        key = (-sum(float(row[i]) for i in sub), sub)
        if best is None or key < best:
            best = key
    return set(best[1])


def brute_expert_side(cands, col, n):
    best = None
    for sub in itertools.combinations(cands, n):
        key = (-sum(float(col[t]) for t in sub), sub)
        if best is None or key < best:
            best = key
    return list(best[1])


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
@pytest.mark.parametrize("seed", range(6))
def test_select_bruteforce(o64, mode, seed):
    rng = np.random.default_rng(100 + seed)
    T, E, k = int(rng.integers(4, 11)), int(rng.integers(2, 5)), 2
    C = int(rng.integers(1, 5))
    # distinct dyadic values: subset sums are exact, so the maximising subset is unique
    delta = (rng.permutation(T * E).reshape(T, E) - T * E / 2) / 64.0
    rt = o64.select(delta, k, mode, C, 8)
    for i in range(E):
        if mode == ob.MODE_TCR:
            cands = [t for t in range(T) if i in brute_token_side(delta[t], k)]
        else:
            cands = list(range(T))
        want = sorted(brute_expert_side(cands, delta[:, i], min(C, len(cands))))
        got = [t for t in rt.slot_token[i * 8:(i + 1) * 8] if t >= 0]
        assert got == want
        assert rt.counts[i] == len(want)
    if mode == ob.MODE_TCR:
        for t in range(T):
            assert set(rt.topk_idx[t]) == brute_token_side(delta[t], k)
            assert delta[t, rt.topk_idx[t, 0]] >= delta[t, rt.topk_idx[t, 1]]


def test_select_tie_breaks(o32):
    delta = np.zeros((6, 3), np.float32)        # everything ties
    rt = o32.select(delta, 2, ob.MODE_TCR, 2, 4)
    assert np.all(rt.topk_idx == np.array([0, 1]))               # lower expert index
    assert list(rt.slot_token[:4]) == [0, 1, -1, -1]             # lower token index
    assert list(rt.slot_token[4:8]) == [0, 1, -1, -1]
    assert rt.counts.tolist() == [2, 2, 0] and rt.dropped == 8 and rt.unrouted == 4
    rt = o32.select(delta, 2, ob.MODE_ECR, 2, 4)
    assert rt.counts.tolist() == [2, 2, 2] and list(rt.slot_token[8:12]) == [0, 1, -1, -1]


def check_route_invariants(delta, rt, k, mode, C, capacity):
    T, E = delta.shape
    Cs = rt.C_stride
    assert C <= capacity <= Cs
    rows_of = [[] for _ in range(T)]
    for i in range(E):
        seg = rt.slot_token[i * Cs:(i + 1) * Cs]
        n = rt.counts[i]
        assert 0 <= n <= C
        assert np.all(seg[:n] >= 0) and np.all(seg[n:] == -1)
        assert np.all(np.diff(seg[:n]) > 0)                      # injective and ascending
        g = rt.gate[i * Cs:(i + 1) * Cs]
        assert np.array_equal(g[:n], delta[seg[:n], i]) and np.all(g[n:] == 0)
        if mode == ob.MODE_TCR:
            cand = np.nonzero((rt.topk_idx == i).any(1))[0]
        else:
            cand = np.arange(T)
            assert n == min(C, T)
        assert n == min(C, len(cand)) and set(seg[:n]) <= set(cand)
        dropped = np.setdiff1d(cand, seg[:n])
        if len(dropped) and n:
            # every dropped candidate ranks no higher than every kept one
            kept_key = min((delta[t, i], -t) for t in seg[:n])
            assert max((delta[t, i], -t) for t in dropped) < kept_key
        for p in range(n):
            rows_of[seg[p]].append(i * Cs + p)
    if mode == ob.MODE_TCR:
        for t in range(T):
            top = rt.topk_idx[t]
            assert len(set(top)) == k
            rest = np.setdiff1d(np.arange(E), top)
            assert np.all(np.diff(delta[t, top]) <= 0)
            if len(rest):
                assert delta[t, top].min() >= delta[t, rest].max()
            assert len(rows_of[t]) <= k and all(r // Cs in top for r in rows_of[t])
    assert rt.tok_ptr[0] == 0 and rt.tok_ptr[T] == rt.counts.sum()
    for t in range(T):
        assert list(rt.tok_row[rt.tok_ptr[t]:rt.tok_ptr[t + 1]]) == rows_of[t]
    assert rt.unrouted == sum(1 for r in rows_of if not r)
    n_cand = T * k if mode == ob.MODE_TCR else T * E
    assert rt.dropped == n_cand - rt.counts.sum()


@pytest.mark.parametrize("name,mode", [("tiny", ob.MODE_TCR), ("tiny", ob.MODE_ECR),
                                       ("small", ob.MODE_TCR), ("mid", ob.MODE_ECR)])
def test_select_invariants(o32, name, mode):
    w = gw.scaled(gw.WORKLOADS[name], T=1024 if name != "tiny" else 512)
    R = gw.expert_embeddings(w)
    X = gw.tokens(w, R)
    delta, *_ = o32.affinity(X, R, D=w.D)
    for C in (w.capacity, max(1, w.capacity // 3)):
        rt = o32.select(delta, w.k, mode, C, w.C_stride)
        check_route_invariants(delta, rt, w.k, mode, C, w.capacity)


def test_select_reductions(o32):
    w = gw.WORKLOADS["tiny"]
    R = gw.expert_embeddings(w)
    X = gw.tokens(w, R)
    delta, *_ = o32.affinity(X, R, D=w.D)
    # capacity >= T in token choice: nothing dropped, k rows per token
    rt = o32.select(delta, w.k, ob.MODE_TCR, w.T, 512)
    assert rt.counts.sum() == w.k * w.T and rt.dropped == 0 and rt.unrouted == 0
    assert np.all(np.diff(rt.tok_ptr) == w.k)
    # k = E in token choice is expert choice
    a = o32.select(delta, w.E, ob.MODE_TCR, 100, 128)
    b = o32.select(delta, w.k, ob.MODE_ECR, 100, 128)
    for f in ("counts", "slot_token", "gate", "tok_ptr", "tok_row"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    # expert choice with C = T: every pair selected
    rt = o32.select(delta, w.k, ob.MODE_ECR, w.T, 512)
    assert np.all(rt.counts == w.T) and np.all(np.diff(rt.tok_ptr) == w.E)


# ------------------------------------------ threshold on the sum of affinity scores ------------
# The rule (a reading of the sentence that introduces the expert-side equation of "Routing
# Strategy": an expert stops taking tokens once their accumulated affinity is large enough) is
# pinned without restating its loop: by exhaustive search over prefix
# lengths in exact rational arithmetic, by its two limits, by a closed form on constant scores and
# by monotonicity in tau.

ROUTE_FIELDS = ("topk_idx", "counts", "slot_token", "gate", "tok_ptr", "tok_row")


def same_route(a, b):
    return all(np.array_equal(getattr(a, f), getattr(b, f)) for f in ROUTE_FIELDS) and \
        a.dropped == b.dropped and a.unrouted == b.unrouted


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
@pytest.mark.parametrize("flags", [1, 2, 3])
def test_threshold_at_infinity_is_the_plain_selection(o32, mode, flags):
    delta = (rand((300, 8), 21) / 16).astype(np.float32)
    for C in (1, 17, 300):
        assert same_route(o32.select(delta, 2, mode, C, 384),
                          o32.select_thresholded(delta, 2, mode, C, 384, flags))


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
def test_threshold_below_the_first_score_keeps_one_and_nonpositive_keeps_none(o32, mode):
    delta = np.abs(rand((200, 6), 22) / 8).astype(np.float32) + np.float32(0.01)      # all positive
    plain1 = o32.select(delta, 2, mode, 1, 128)              # capacity 1: each expert's best candidate
    tiny = o32.select_thresholded(delta, 2, mode, 50, 128, 1, tau_expert=1e-6)
    assert np.array_equal(tiny.counts, plain1.counts) and np.array_equal(tiny.slot_token, plain1.slot_token)
    for tau in (0.0, -1.0):
        none = o32.select_thresholded(delta, 2, mode, 50, 128, 1, tau_expert=tau)
        assert np.all(none.counts == 0) and none.unrouted == 200 and none.tok_ptr[-1] == 0
    # token side: a token whose first affinity already reaches tau takes that expert only
    one = o32.select_thresholded(delta, 3, ob.MODE_TCR, 200, 256, 2, tau_token=1e-6)
    top = o32.select(delta, 1, ob.MODE_TCR, 200, 256)
    assert np.array_equal(one.topk_idx[:, 0], top.topk_idx[:, 0]) and np.all(one.topk_idx[:, 1:] == -1)
    assert np.array_equal(one.counts, top.counts) and np.array_equal(one.slot_token, top.slot_token)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
def test_threshold_bruteforce_over_prefixes(o64, mode, seed):
    """Scores are multiples of 1/64, so sums are exact both as 2^-32 integers and as fractions.
    For every expert, among all prefix lengths n of its candidate list in (score descending, token
    ascending) order, the answer is the longest n <= C all of whose proper prefixes (lengths
    0..n-1) sum to less than tau."""
    from fractions import Fraction
    rng = np.random.default_rng(100 + seed)
    T, E, k, C = 12, 3, 2, 7
    delta = rng.integers(-20, 40, size=(T, E)) / 64.0
    tau = Fraction(int(rng.integers(1, 200)), 64)
    got = o64.select_thresholded(delta, k, mode, C, 128, 1, tau_expert=float(tau))
    plain = o64.select(delta, k, mode, T, 128)               # no cut: each expert's full candidate list
    for i in range(E):
        cand = plain.slot_token[i * 128:i * 128 + plain.counts[i]]
        order = sorted(cand, key=lambda t: (-delta[t, i], t))
        best = 0
        for n in range(0, min(C, len(order)) + 1):
            sums = [sum((Fraction(delta[t, i]) for t in order[:j]), Fraction(0)) for j in range(n)]
            if all(s < tau for s in sums):
                best = n
        assert got.counts[i] == best
        assert sorted(order[:best]) == list(got.slot_token[i * 128:i * 128 + best])
    if mode == ob.MODE_TCR:      # token side, same search over each token's ranked experts (k = 3, mixed signs)
        tok = o64.select_thresholded(delta, 3, mode, T, 128, 2, tau_token=float(tau))
        for t in range(T):
            order = sorted(range(E), key=lambda i: (-delta[t, i], i))
            best = 0
            for n in range(0, 4):
                sums = [sum((Fraction(delta[t, i]) for i in order[:j]), Fraction(0)) for j in range(n)]
                if all(s < tau for s in sums):
                    best = n
            assert list(tok.topk_idx[t]) == order[:best] + [-1] * (3 - best)


def test_threshold_closed_form_on_constant_scores(o32):
    """All affinities equal to a = 1/8: an expert keeps min(C, T, ceil(tau / a)) tokens, lowest ids first."""
    T, E, C = 40, 4, 30
    delta = np.full((T, E), 0.125, np.float32)
    for tau, want in ((0.1, 1), (0.125, 1), (0.126, 2), (1.0, 8), (1.01, 9), (3.75, 30), (100.0, 30)):
        r = o32.select_thresholded(delta, 2, ob.MODE_ECR, C, 128, 1, tau_expert=tau)
        assert np.all(r.counts == want), (tau, r.counts)
        assert np.array_equal(r.slot_token[:want], np.arange(want))
    # token side, k = 4 experts of affinity 1/8 each: ceil(tau / a) experts, capped by k
    for tau, want in ((0.125, 1), (0.2, 2), (0.4, 4), (9.0, 4)):
        r = o32.select_thresholded(delta, 4, ob.MODE_TCR, T, 128, 2, tau_token=tau)
        assert np.all((r.topk_idx >= 0).sum(1) == want)
        assert np.array_equal(r.topk_idx[0, :want], np.arange(want))


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
def test_threshold_is_monotone_and_keeps_a_prefix(o32, mode):
    delta = (rand((500, 8), 23) / 12).astype(np.float32)     # mixed signs
    C, Cs = 90, 128
    prev = None
    full = o32.select(delta, 2, mode, 500, 512)
    for tau in (0.05, 0.3, 1.0, 2.5, 6.0, 1e9):
        r = o32.select_thresholded(delta, 2, mode, C, Cs, 1, tau_expert=tau)
        assert np.all(r.counts <= C)
        for i in range(8):
            kept = set(r.slot_token[i * Cs:i * Cs + r.counts[i]])
            cand = full.slot_token[i * 512:i * 512 + full.counts[i]]
            order = sorted(cand, key=lambda t: (-delta[t, i], t))
            assert kept == set(order[:r.counts[i]])          # a prefix of the ranked candidates
            if prev is not None:
                assert prev[i] <= kept                       # grows with tau
        prev = [set(r.slot_token[i * Cs:i * Cs + r.counts[i]]) for i in range(8)]
    assert same_route(r, o32.select(delta, 2, mode, C, Cs))  # a huge tau is no cut at all


def test_threshold_sum_does_not_depend_on_float_summation_order(o32):
    """Scores whose float sum depends on the order (1/3-like values of mixed size): the decision is
    taken on 2^-32 integers, so it equals the one computed with Python integers."""
    rng = np.random.default_rng(9)
    T = 4000
    delta = (rng.random((T, 1)) * 0.3 + 1e-4).astype(np.float32)
    tau = 57.123
    r = o32.select_thresholded(delta, 1, ob.MODE_ECR, T, 4096, 1, tau_expert=tau)
    q = [int(round(float(v) * 2 ** 32)) for v in delta[:, 0]]          # exact: float * 2^32 is an integer or a dyadic
    order = sorted(range(T), key=lambda t: (-q[t], t))
    tq, s, n = int(round(tau * 2 ** 32)), 0, 0
    while n < T and s < tq:
        s += q[order[n]]
        n += 1
    assert r.counts[0] == n
