"""Parity of the CUDA path (through the C ABI) against the CPU oracle, stage by stage and
for the whole layer, at sizes the oracle finishes in seconds.  The sizes span several
tiles of every kernel and leave ragged tails (T not a multiple of 32, h not a multiple of
128, per-expert row counts not multiples of 128).

Tolerances (from the target statement):
  affinities          |err| <= 1e-5 * max(|ref|, rms(ref))           (fp32)
  routing             bit-exact wherever the oracle's score margin exceeds 1e-5; with the
                      oracle's own affinities as input, bit-exact everywhere
  outputs, gradients  max|err| <= 2e-2 * rms(ref tensor) for bf16 storage / fp32 accumulate,
                      1e-4 * rms for the fp32 layer
"""
import numpy as np
import pytest
import torch

from gen import workloads as gw
from oracle import binding as ob
from tests import harness as hz

pytestmark = pytest.mark.gpu

etr = hz.etr

W = gw.WORKLOADS
CASES = {
    "tiny": W["tiny"],
    "tiny_ecr": gw.scaled(W["tiny"], name="tiny_ecr", mode="ecr", cf=1.0),
    "small_s": gw.scaled(W["small"], name="small_s", T=1000, d=512, D=8, E=16, h=320),
    "mid_s": gw.scaled(W["mid"], name="mid_s", T=1536, d=512, D=8, E=8, h=384, n_clusters=8),
    # d = 2048: 4 KiB token rows and 256 pooled columns, as in the mid and sweep workloads
    "mid_w": gw.scaled(W["mid"], name="mid_w", T=1500, d=2048, D=8, E=8, h=128, n_clusters=32),
    "sweep_s_tcr": gw.scaled(W["sweep"], name="sweep_s_tcr", T=2048, d=1024, D=16, E=16, h=256,
                             n_clusters=16, step=600),
    "sweep_s_ecr": gw.scaled(W["sweep"], name="sweep_s_ecr", T=2048, d=1024, D=16, E=16, h=256,
                             n_clusters=16, step=1500),
}
SWEEP_OVERRIDE = 0.125      # puts the adaptive bound inside (c_floor, capacity) for d=1024, E=16


def rel_tol(w):
    return 2e-2 if w.dtype == "bf16" else 1e-4


def override_of(name):
    return SWEEP_OVERRIDE if name.startswith("sweep") else -1.0


_cache = {}


def case(name):
    """Inputs, oracle forward and backward of a case (cached per session)."""
    if name not in _cache:
        w = CASES[name]
        inp = gw.make_inputs(w)
        o = ob.Oracle("f32")
        fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k,
                       capacity=w.capacity, mode=hz.mode_of(w), adaptive=w.adaptive,
                       delta_max_override=override_of(name))
        bw = o.backward(fw, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
        _cache[name] = (w, inp, o, fw, bw)
    return _cache[name]


@pytest.mark.parametrize("name", list(CASES))
def test_affinity(name):
    w, inp, o, fw, _ = case(name)
    cfg = hz.make_cfg(w)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    buf.stats.zero_()
    etr.affinity(cfg, dev.X, dev.R, buf.delta, buf.Z, buf.xnorm, buf.rnorm, buf.c.stats)
    torch.cuda.synchronize()
    hz.assert_affinity_close(hz.to_np(buf.delta), fw.delta)
    assert np.allclose(hz.to_np(buf.xnorm), fw.xnorm, rtol=2e-6, atol=0)
    assert np.allclose(hz.to_np(buf.rnorm), fw.rnorm, rtol=2e-6, atol=0)
    assert int(buf.stats[5].item()) & 0xffffffff == etr_key(hz.to_np(buf.delta).max())
    zref = inp["X"].reshape(w.T, w.m, w.D).astype(np.float64).mean(-1)
    assert np.allclose(hz.to_np(buf.Z), zref, rtol=1e-5, atol=1e-6)


def run_select(w, cfg, delta_np):
    buf = etr.LayerBuffers(cfg)
    buf.stats.zero_()
    buf.delta.copy_(torch.from_numpy(delta_np))
    buf.stats[5] = int(np.array([etr_key(delta_np.max())], dtype=np.uint32).view(np.int32)[0])
    ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    etr.select(cfg, buf.delta, buf.c.stats, buf.route, ws)
    torch.cuda.synchronize()
    return buf, hz.route_from_buffers(buf, cfg)


def etr_key(f):
    u = int(np.float32(f).view(np.uint32))
    return (~u & 0xffffffff) if (u & 0x80000000) else (u | 0x80000000)


def routes_equal(a, b):
    n = a.tok_ptr[-1]
    return (a.C == b.C and np.array_equal(a.counts, b.counts)
            and np.array_equal(a.slot_token, b.slot_token) and np.array_equal(a.gate, b.gate)
            and np.array_equal(a.tok_ptr, b.tok_ptr) and np.array_equal(a.tok_row[:n], b.tok_row[:n])
            and np.array_equal(a.topk_idx, b.topk_idx) and a.dropped == b.dropped
            and a.unrouted == b.unrouted)


@pytest.mark.parametrize("name", list(CASES))
def test_select_bit_exact_on_oracle_affinities(name):
    """Same affinity bits in, so every index, count and map must be identical."""
    w, inp, o, fw, _ = case(name)
    cfg = hz.make_cfg(w, delta_max_override=override_of(name))
    buf, got = run_select(w, cfg, fw.delta)
    assert routes_equal(fw.route, got)
    if name.startswith("sweep"):
        assert 1 < got.C < w.capacity        # the adaptive bound is in the interior of its clamp
    hz.check_route_structure(fw.delta, got, hz.mode_of(w))


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
@pytest.mark.parametrize("capacity", [1, 37, 128, 300])
def test_select_capacities_and_modes(mode, capacity):
    w = gw.scaled(W["tiny"], T=777, cf=(capacity - 0.5) * 8 / (777 * 2))
    assert w.capacity == capacity
    inp = gw.make_inputs(w, weights=False)
    o = ob.Oracle("f32")
    delta, *_ = o.affinity(inp["X"], inp["R"], w.D)
    ref = o.select(delta, w.k, mode, capacity, w.C_stride)
    cfg = hz.make_cfg(w, mode=mode)
    _, got = run_select(w, cfg, delta)
    assert routes_equal(ref, got)


@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
def test_select_ties_go_to_lower_index(mode):
    """Heavily tied affinities (few distinct values): the tie-break decides almost everything."""
    w = gw.scaled(W["tiny"], T=600, cf=0.5)
    rng = np.random.default_rng(7)
    delta = (rng.integers(-2, 3, size=(w.T, w.E)) / 8.0).astype(np.float32)
    o = ob.Oracle("f32")
    ref = o.select(delta, w.k, mode, w.capacity, w.C_stride)
    _, got = run_select(w, hz.make_cfg(w, mode=mode), delta)
    assert routes_equal(ref, got)
    delta[:] = 0.25
    ref = o.select(delta, w.k, mode, w.capacity, w.C_stride)
    _, got = run_select(w, hz.make_cfg(w, mode=mode), delta)
    assert routes_equal(ref, got)


@pytest.mark.parametrize("name", ["tiny", "small_s", "mid_s"])
def test_dispatch_combine_and_backward(name):
    w, inp, o, fw, bw = case(name)
    cfg = hz.make_cfg(w)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    hz.upload_route(buf, fw.route)
    # dispatch: bit-exact copy; pad rows zero
    buf.Xp.fill_(float("nan"))
    etr.dispatch(cfg, dev.X, buf.route, buf.Xp)
    Xp = hz.to_np(buf.Xp)
    Cs = w.C_stride
    for i in range(w.E):
        lim = (fw.route.counts[i] + 127) // 128 * 128
        assert np.array_equal(Xp[i * Cs:i * Cs + lim], fw.Xp[i * Cs:i * Cs + lim])
        assert np.isnan(Xp[i * Cs + lim:(i + 1) * Cs]).all()
    # combine on the oracle's O
    buf.O.copy_(hz.to_dev(fw.O, w))
    O_grid = hz.to_np(buf.O)
    Y = torch.empty_like(dev.X)
    etr.combine(cfg, buf.route, buf.O, Y)
    hz.assert_close_rms(hz.to_np(Y), o.combine(O_grid, fw.route), rel_tol(w), "Y")
    # combine backward
    etr.combine_bwd(cfg, buf.route, dev.dY, buf.O, buf.dO, buf.dgate)
    dO_ref, dgate_ref = o.combine_bwd(inp["dY"], O_grid, fw.route)
    used = (np.arange(Cs)[None, :] < ((fw.route.counts + 127) // 128 * 128)[:, None]).reshape(-1)
    hz.assert_close_rms(hz.to_np(buf.dO)[used], dO_ref[used], rel_tol(w), "dO")
    hz.assert_close_rms(hz.to_np(buf.dgate)[used], dgate_ref[used], 1e-4, "dgate")
    # dispatch backward
    buf.dXp.copy_(hz.to_dev(bw.dXp, w))
    dX = torch.empty_like(dev.X)
    etr.dispatch_bwd(cfg, buf.route, buf.dXp, dX)
    hz.assert_close_rms(hz.to_np(dX), o.dispatch_bwd(hz.to_np(buf.dXp), fw.route), rel_tol(w), "dX_ffn")


def ffn_stage(name, impl):
    w, inp, o, fw, bw = case(name)
    cfg = hz.make_cfg(w, gemm_impl=impl)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    hz.upload_route(buf, fw.route)
    buf.stats.zero_()
    tol = rel_tol(w)
    etr.dispatch(cfg, dev.X, buf.route, buf.Xp)
    for t in (buf.G, buf.U, buf.H, buf.O):
        t.fill_(float("nan"))
    ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    etr.expert_ffn(cfg, buf.route, buf.Xp, dev.W1g, dev.W1u, dev.W2, buf.G, buf.U, buf.H, buf.O,
                   buf.c.stats, ws)
    Cs = w.C_stride
    used = (np.arange(Cs)[None, :] < fw.route.counts[:, None]).reshape(-1)
    padded = (np.arange(Cs)[None, :] < ((fw.route.counts + 127) // 128 * 128)[:, None]).reshape(-1)
    for nm in ("G", "U", "H", "O"):
        got = hz.to_np(getattr(buf, nm))
        hz.assert_close_rms(got[used], getattr(fw, nm)[used], tol, nm, chain=2 if nm == "O" else 1)
        assert np.all(got[padded & ~used] == 0), f"{nm}: pad rows must be zero"
    # Backward as a stage of its own: every input is the oracle's, rounded to the storage
    # grid, and the oracle is run on exactly those rounded values.
    grid = (lambda a: gw.round_to_bf16(a)) if w.dtype == "bf16" else (lambda a: a)
    dOq, Gq, Uq, Hq = grid(bw.dO), grid(fw.G), grid(fw.U), grid(fw.H)
    for nm, a in (("dO", dOq), ("G", Gq), ("U", Uq), ("H", Hq)):
        getattr(buf, nm).copy_(hz.to_dev(a, w))
    ref = o.expert_ffn_bwd(dOq, fw.Xp, Gq, Uq, Hq, fw.route, inp["W1g"], inp["W1u"], inp["W2"])
    r_dG, r_dU, r_dXp, r_dW1g, r_dW1u, r_dW2 = ref
    dW1g, dW1u, dW2 = (torch.full_like(t, float("nan")) for t in (dev.W1g, dev.W1u, dev.W2))
    etr.expert_ffn_bwd(cfg, buf.route, buf.dO, buf.Xp, buf.G, buf.U, buf.H, dev.W1g, dev.W1u, dev.W2,
                       buf.dG, buf.dU, buf.dXp, dW1g, dW1u, dW2, buf.c.stats, ws)
    assert buf.read_stats().error_word == 0
    hz.assert_close_rms(hz.to_np(buf.dG)[used], r_dG[used], tol, "dG")
    hz.assert_close_rms(hz.to_np(buf.dU)[used], r_dU[used], tol, "dU")
    # dXp and dW1* consume the kernel's own bf16 dG and dU (two more stored tensors)
    hz.assert_close_rms(hz.to_np(buf.dXp)[used], r_dXp[used], tol, "dXp", chain=3)
    hz.assert_close_rms(hz.to_np(dW1g), r_dW1g, tol, "dW1g", chain=3)
    hz.assert_close_rms(hz.to_np(dW1u), r_dW1u, tol, "dW1u", chain=3)
    hz.assert_close_rms(hz.to_np(dW2), r_dW2, tol, "dW2", chain=2)


@pytest.mark.parametrize("name", ["tiny", "tiny_ecr", "small_s", "mid_s"])
def test_expert_ffn_simt(name):
    ffn_stage(name, etr.GEMM_SIMT)


@pytest.mark.parametrize("name", ["small_s", "mid_s", "sweep_s_tcr", "sweep_s_ecr"])
def test_expert_ffn_tcgen05(name):
    ffn_stage(name, etr.GEMM_TCGEN05)


@pytest.mark.parametrize("name", ["small_s", "mid_s", "sweep_s_tcr", "sweep_s_ecr"])
def test_expert_ffn_tcgen05_two_cta(name):
    ffn_stage(name, etr.GEMM_TCGEN05_2CTA)


@pytest.mark.parametrize("name", ["small_s", "mid_s", "sweep_s_tcr", "sweep_s_ecr"])
def test_expert_ffn_tcgen05_two_cta_wide(name):
    ffn_stage(name, etr.GEMM_TCGEN05_2CTA_WIDE)


def run_layer(w, inp, cfg, host_step=False):
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg, host_staging=host_step)
    out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
               dW1g=torch.empty_like(dev.W1g), dW1u=torch.empty_like(dev.W1u),
               dW2=torch.empty_like(dev.W2))
    if host_step:
        Xh, dYh = dev.X.cpu().pin_memory(), dev.dY.cpu().pin_memory()
        Yh, dXh = torch.empty_like(Xh).pin_memory(), torch.empty_like(Xh).pin_memory()
        etr.layer_step_host(cfg, Xh, dYh, dev.R, dev.W1g, dev.W1u, dev.W2, buf, Yh, dXh, out["dR"],
                            out["dW1g"], out["dW1u"], out["dW2"])
        out["Y"], out["dX"] = Yh, dXh
    else:
        etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
        etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"],
                           out["dR"], out["dW1g"], out["dW1u"], out["dW2"])
    torch.cuda.synchronize()
    return buf, out


@pytest.mark.parametrize("name", list(CASES))
def test_layer_forward_backward(name):
    w, inp, o, fw, bw = case(name)
    # capacity parity: the device takes the oracle's delta_max so both sides clamp the same C
    ov = override_of(name) if w.adaptive else -1.0
    cfg = hz.make_cfg(w, delta_max_override=ov)
    buf, out = run_layer(w, inp, cfg)
    st = buf.read_stats()
    assert st.error_word == 0
    assert abs(st.delta_max - float(fw.delta_max)) <= 1e-5 * abs(float(fw.delta_max))
    got = hz.route_from_buffers(buf, cfg)
    delta_dev = hz.to_np(buf.delta)
    hz.assert_affinity_close(delta_dev, fw.delta)
    hz.check_route_structure(delta_dev, got, hz.mode_of(w))
    identical = hz.assert_routes_match(fw.delta, fw.route, got, hz.mode_of(w))
    if not identical:      # margin-exempt differences: compare values on the device's own route
        fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k,
                       capacity=w.capacity, route=got)
        bw = o.backward(fw, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    # bf16 tensors stored on the path to each output (see assert_close_rms):
    #   Y: Xp, H, O, Y                        dW2: dO, H, Xp (through H), dW2
    #   dX: dO, G, U, dG|dU, dXp, dX          dW1*: dO, G, U, dG|dU, Xp, dW1
    tol = rel_tol(w)
    hz.assert_close_rms(hz.to_np(out["Y"]), fw.Y, tol, "Y", chain=4)
    hz.assert_close_rms(hz.to_np(out["dX"]), bw.dX, tol, "dX", chain=6)
    hz.assert_close_rms(hz.to_np(out["dR"]), bw.dR, tol, "dR", chain=4)
    hz.assert_close_rms(hz.to_np(out["dW1g"]), bw.dW1g, tol, "dW1g", chain=6)
    hz.assert_close_rms(hz.to_np(out["dW1u"]), bw.dW1u, tol, "dW1u", chain=6)
    hz.assert_close_rms(hz.to_np(out["dW2"]), bw.dW2, tol, "dW2", chain=4)


def test_layer_is_deterministic_and_host_step_matches():
    w, inp, o, fw, bw = case("small_s")
    cfg = hz.make_cfg(w)
    _, a = run_layer(w, inp, cfg)
    _, b = run_layer(w, inp, cfg)
    _, c = run_layer(w, inp, cfg, host_step=True)
    for k in a:
        assert torch.equal(a[k], b[k]), k
        assert torch.equal(a[k].cpu(), c[k].cpu()), k


@pytest.mark.parametrize("impl", [etr.GEMM_AUTO, etr.GEMM_TCGEN05_2CTA, etr.GEMM_TCGEN05_2CTA_WIDE])
@pytest.mark.parametrize("name", ["small_s", "mid_s", "sweep_s_tcr", "sweep_s_ecr"])
def test_fused_dispatch_gives_the_same_bits(name, impl):
    """With the token rearrangement fused into the operand fetch (TMA row gathers from X) the GEMMs
    see the same operands in the same order: every output must equal the unfused path bit for bit,
    and Xp must not have been touched."""
    w, inp, o, fw, bw = case(name)
    ov = override_of(name) if w.adaptive else -1.0
    _, ref = run_layer(w, inp, hz.make_cfg(w, gemm_impl=impl, delta_max_override=ov, fuse_dispatch=etr.FUSE_OFF))
    cfg = hz.make_cfg(w, gemm_impl=impl, delta_max_override=ov, fuse_dispatch=etr.FUSE_ON)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    buf.Xp.fill_(float("nan"))
    out = {k: torch.empty_like(v) for k, v in ref.items()}
    etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
    etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                       out["dW1g"], out["dW1u"], out["dW2"])
    torch.cuda.synchronize()
    assert buf.read_stats().error_word == 0
    assert bool(torch.isnan(buf.Xp).all()), "Xp was written"
    for k in ref:
        assert torch.equal(out[k], ref[k]), k


@pytest.mark.parametrize("name", ["tiny", "small_s", "mid_s"])
def test_softmax_gate_stages_and_load_stats(name):
    """etr_gate_softmax, etr_gate_softmax_bwd, etr_affinity_bwd_dense and etr_load_stats one by one,
    each fed with the oracle's inputs of that stage (fp32 routing tensors: 1e-5-level agreement)."""
    w, inp, o, fw, bw = case(name)
    cfg = hz.make_cfg(w, gate_mode=etr.GATE_SOFTMAX)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    hz.upload_route(buf, fw.route)
    buf.delta.copy_(torch.from_numpy(fw.delta))
    rt = fw.route
    rows = np.nonzero(rt.slot_token >= 0)[0]
    # forward: gates and log-sum-exp (library: torch.logsumexp in float64)
    etr.gate_softmax(cfg, buf.delta, buf.route, buf.lse)
    gate_ref = o.softmax_gate(fw.delta, rt)
    got_gate = hz.to_np(buf.gate)
    assert np.allclose(got_gate[rows], gate_ref[rows], rtol=2e-6, atol=0)
    assert np.all(got_gate[rt.slot_token < 0] == 0)
    lse_ref = torch.logsumexp(torch.from_numpy(fw.delta).double(), dim=1).numpy()
    assert np.allclose(hz.to_np(buf.lse), lse_ref, rtol=1e-6, atol=1e-6)
    # load statistics of the softmax gates and of the raw gates
    load, gm = torch.empty(w.E, device="cuda"), torch.empty(w.E, device="cuda")
    etr.load_stats(cfg, buf.route, load, gm)
    l_ref, g_ref = o.load_stats(rt, gate_ref)
    assert np.array_equal(hz.to_np(load), l_ref) and np.allclose(hz.to_np(gm), g_ref, rtol=1e-5, atol=1e-9)
    # backward of the gate: dense d delta from the oracle's dgate (of the raw-gate backward pass:
    # any dgate serves here)
    buf.dgate.copy_(torch.from_numpy(bw.dgate))
    etr.gate_softmax_bwd(cfg, buf.delta, buf.lse, buf.route, buf.dgate, buf.ddelta)
    dd_ref = o.softmax_gate_bwd(fw.delta, bw.dgate, rt)
    hz.assert_close_rms(hz.to_np(buf.ddelta), dd_ref, 1e-4, "ddelta")
    unrouted = np.diff(rt.tok_ptr) == 0
    assert np.all(hz.to_np(buf.ddelta)[unrouted] == 0)
    # dense router gradient on the oracle's d delta
    buf.ddelta.copy_(torch.from_numpy(dd_ref))
    etr.affinity(cfg, dev.X, dev.R, buf.delta, buf.Z, buf.xnorm, buf.rnorm, buf.c.stats)
    base = (np.arange(w.T * w.d, dtype=np.float32).reshape(w.T, w.d) % 7 - 3) / 4     # exact in bf16
    dX = hz.to_dev(base, w)
    dR = torch.empty_like(dev.R)
    ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    etr.affinity_bwd_dense(cfg, dev.X, dev.R, buf.delta, buf.Z, buf.xnorm, buf.rnorm, buf.route, buf.ddelta,
                           dX, dR, ws)
    dX_ref, dR_ref = o.affinity_bwd(inp["X"], inp["R"], w.D, fw.delta, fw.xnorm, fw.rnorm, dd_ref, base.copy())
    hz.assert_close_rms(hz.to_np(dX), dX_ref, rel_tol(w), "dX (dense router term)")
    hz.assert_close_rms(hz.to_np(dR), dR_ref, 1e-4, "dR (dense)")


@pytest.mark.parametrize("name", ["tiny", "small_s", "mid_s", "sweep_s_tcr", "sweep_s_ecr"])
def test_layer_with_softmax_gate(name):
    """Whole layer with the softmax gate against the oracle, fp32 and bf16, both selection modes."""
    w, inp, o, _, _ = case(name)
    ov = override_of(name)
    fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k, capacity=w.capacity,
                   mode=hz.mode_of(w), adaptive=w.adaptive, delta_max_override=ov, softmax_gate=True)
    bw = o.backward(fw, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    cfg = hz.make_cfg(w, delta_max_override=ov if w.adaptive else -1.0, gate_mode=etr.GATE_SOFTMAX)
    buf, out = run_layer(w, inp, cfg)
    assert buf.read_stats().error_word == 0
    got = hz.route_from_buffers(buf, cfg)
    assert hz.assert_routes_match(fw.delta, fw.route, got, hz.mode_of(w)), "cases with clear margins"
    rows = np.nonzero(got.slot_token >= 0)[0]
    assert np.allclose(got.gate[rows], fw.gate[rows], rtol=1e-5, atol=0)
    tol = rel_tol(w)
    hz.assert_close_rms(hz.to_np(out["Y"]), fw.Y, tol, "Y", chain=4)
    hz.assert_close_rms(hz.to_np(out["dX"]), bw.dX, tol, "dX", chain=6)
    hz.assert_close_rms(hz.to_np(out["dR"]), bw.dR, tol, "dR", chain=4)
    frac = hz.dw1_outlier_fraction(w)      # clustered tokens: see harness.OUTLIER_FRACTION_CLUSTERED_DW1
    hz.assert_close_rms(hz.to_np(out["dW1g"]), bw.dW1g, tol, "dW1g", chain=6, outlier_fraction=frac)
    hz.assert_close_rms(hz.to_np(out["dW1u"]), bw.dW1u, tol, "dW1u", chain=6, outlier_fraction=frac)
    hz.assert_close_rms(hz.to_np(out["dW2"]), bw.dW2, tol, "dW2", chain=4)


def test_pipelined_host_steps_match_the_layer_calls():
    """Six steps through etr_layer_step_host_begin on two slots, alternating between two different
    batches, with no wait between them: every step must deliver exactly what the layer calls give
    for its own batch (slots do not leak into each other, re-use of a slot is ordered)."""
    w, inp, o, fw, bw = case("small_s")
    cfg = hz.make_cfg(w)
    inp2 = dict(inp)
    inp2["X"] = np.ascontiguousarray(inp["X"][::-1])          # another batch: the tokens reversed
    inp2["dY"] = np.ascontiguousarray(inp["dY"][::-1] * 0.5)
    refs = [run_layer(w, q, cfg)[1] for q in (inp, inp2)]
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    slots = [etr.HostSlot(cfg, i) for i in range(2)]
    host = []
    for q in (inp, inp2):
        d = hz.upload(w, q)
        host.append((d.X.cpu().pin_memory(), d.dY.cpu().pin_memory()))
    outs = [(torch.empty_like(host[0][0]).pin_memory(), torch.empty_like(host[0][0]).pin_memory())
            for _ in range(6)]
    g = dict(dR=torch.empty_like(dev.R), dW1g=torch.empty_like(dev.W1g), dW1u=torch.empty_like(dev.W1u),
             dW2=torch.empty_like(dev.W2))
    for i in range(6):
        Xh, dYh = host[i % 2]
        etr.layer_step_host_begin(cfg, Xh, dYh, dev.R, dev.W1g, dev.W1u, dev.W2, buf, slots[i % 2],
                                  outs[i][0], outs[i][1], g["dR"], g["dW1g"], g["dW1u"], g["dW2"])
    for sl in slots:
        etr.layer_step_host_wait(sl)
    torch.cuda.synchronize()
    for i in range(6):
        assert torch.equal(outs[i][0], refs[i % 2]["Y"].cpu()), ("Y", i)
        assert torch.equal(outs[i][1], refs[i % 2]["dX"].cpu()), ("dX", i)
    for k in g:                                               # the last step used the second batch
        assert torch.equal(g[k], refs[1][k]), k
    with pytest.raises(etr.EtrError):
        etr.layer_step_host_wait(etr.HostSlot(cfg, etr.HOST_SLOTS))


@pytest.mark.parametrize("name", ["tiny", "small_s", "mid_s", "mid_w"])
def test_stage_calls_compose_to_the_layer_calls(name):
    """The ten stage entry points called one by one give what etr_layer_forward/backward give.
    Only dX may differ, by one rounding: the layer call fuses the dispatch backward into the
    router-gradient kernel and keeps the row sum in fp32, the stage path stores it first."""
    w, inp, o, fw, bw = case(name)
    cfg = hz.make_cfg(w)
    dev = hz.upload(w, inp)
    _, ref = run_layer(w, inp, cfg)
    buf = etr.LayerBuffers(cfg)
    ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    out = {k: torch.empty_like(v) for k, v in ref.items()}
    buf.stats.zero_()
    etr.affinity(cfg, dev.X, dev.R, buf.delta, buf.Z, buf.xnorm, buf.rnorm, buf.c.stats)
    etr.select(cfg, buf.delta, buf.c.stats, buf.route, ws)
    etr.dispatch(cfg, dev.X, buf.route, buf.Xp)
    etr.expert_ffn(cfg, buf.route, buf.Xp, dev.W1g, dev.W1u, dev.W2, buf.G, buf.U, buf.H, buf.O, buf.c.stats, ws)
    etr.combine(cfg, buf.route, buf.O, out["Y"])
    etr.combine_bwd(cfg, buf.route, dev.dY, buf.O, buf.dO, buf.dgate)
    etr.expert_ffn_bwd(cfg, buf.route, buf.dO, buf.Xp, buf.G, buf.U, buf.H, dev.W1g, dev.W1u, dev.W2,
                       buf.dG, buf.dU, buf.dXp, out["dW1g"], out["dW1u"], out["dW2"], buf.c.stats, ws)
    etr.dispatch_bwd(cfg, buf.route, buf.dXp, out["dX"])
    etr.select_bwd(cfg, buf.route, buf.dgate)
    etr.affinity_bwd(cfg, dev.X, dev.R, buf.delta, buf.Z, buf.xnorm, buf.rnorm, buf.route, buf.dgate,
                     out["dX"], out["dR"], ws)
    torch.cuda.synchronize()
    for k in ("Y", "dR", "dW1g", "dW1u", "dW2"):
        assert torch.equal(out[k], ref[k]), k
    a, b = hz.to_np(out["dX"]), hz.to_np(ref["dX"])
    if w.dtype == "bf16":      # one extra bf16 rounding of a sum that may cancel
        hz.assert_close_rms(a, b, 1e-2, "dX (stage path vs fused)", chain=2)
    else:
        assert np.allclose(a, b, rtol=1e-6, atol=1e-7)


@pytest.mark.parametrize("gate", ["affinity", "softmax"])
@pytest.mark.parametrize("name", ["small_s", "mid_s", "mid_w", "sweep_s_tcr", "sweep_s_ecr"])
def test_parity_with_the_storage_grid_modelled(name, gate):
    """The sharp version of the value comparison, with no exceptions: every stored activation and
    every output and gradient of the layer against the oracle's stages composed with the same
    bf16 roundings the CUDA path applies when it stores G, U, H, O, Y, dO, dG, dU, dXp, dX and the
    weight gradients (harness.storage_grid_reference).  What is left between the two sides is
    fp32-vs-double summation order and the odd flip of a final rounding.  G, U, H and dO (computed
    from exact inputs) must agree to one bf16 ulp of the element plus 2e-4 of the RMS; everything
    downstream of a stored tensor to the target's bound, 2e-2 of the RMS, plus the element's own
    last-bit flip (dG and dU, elementwise products of the stored G and U, also carry the flips of
    those factors)."""
    w, inp, o, fw, bw = case(name)
    soft = gate == "softmax"
    ov = override_of(name)
    if soft:
        fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k, capacity=w.capacity,
                       mode=hz.mode_of(w), adaptive=w.adaptive, delta_max_override=ov, softmax_gate=True)
    cfg = hz.make_cfg(w, delta_max_override=ov if w.adaptive else -1.0,
                      gate_mode=etr.GATE_SOFTMAX if soft else etr.GATE_AFFINITY)
    buf, out = run_layer(w, inp, cfg)
    assert buf.read_stats().error_word == 0
    got = hz.route_from_buffers(buf, cfg)
    assert hz.assert_routes_match(fw.delta, fw.route, got, hz.mode_of(w)), "these cases have clear margins"
    rt = fw.route
    ref = hz.storage_grid_reference(o, w, inp, fw, softmax_gate=soft)
    used = (np.arange(w.C_stride)[None, :] < rt.counts[:, None]).reshape(-1)
    routed = np.diff(rt.tok_ptr) > 0                  # unrouted tokens are exact zeros on both sides
    for nm in ("G", "U", "H", "dO"):
        hz.assert_on_grid(hz.to_np(getattr(buf, nm))[used], getattr(ref, nm)[used], nm, rms_rel=2e-4)
    hz.assert_on_grid(hz.to_np(buf.O)[used], ref.O[used], "O")
    hz.assert_on_grid(hz.to_np(buf.dG)[used], ref.dG[used], "dG", ulps=3)
    hz.assert_on_grid(hz.to_np(buf.dU)[used], ref.dU[used], "dU", ulps=2)
    hz.assert_on_grid(hz.to_np(buf.dXp)[used], ref.dXp[used], "dXp")
    hz.assert_within(hz.to_np(buf.dgate)[used], ref.dgate[used], 1e-2, "dgate vs grid")
    assert np.all(hz.to_np(out["Y"])[~routed] == 0) and np.all(hz.to_np(out["dX"])[~routed] == 0)
    # Y and dX are sums of a token's few stored rows (O, dXp): the flips of those rows arrive undiluted
    for nm in ("Y", "dX"):
        hz.assert_on_grid(hz.to_np(out[nm]), getattr(ref, nm), nm, ulps=2)
    for nm in ("dW1g", "dW1u", "dW2"):
        hz.assert_on_grid(hz.to_np(out[nm]), getattr(ref, nm), nm)
    hz.assert_within(hz.to_np(out["dR"]), ref.dR, 1e-2, "dR vs grid")


def test_argument_errors_are_reported_without_launching():
    import ctypes as C
    w = CASES["tiny"]
    good = hz.make_cfg(w)
    assert etr.validate(good) == etr.OK
    n0 = etr.launch_count()
    bad = hz.make_cfg(gw.scaled(w, D=3))
    assert etr.validate(bad) == etr.ERR_SHAPE
    assert etr.validate(hz.make_cfg(gw.scaled(w, k=9))) == etr.ERR_SHAPE
    assert etr.validate(hz.make_cfg(gw.scaled(w, E=128, D=4))) == etr.ERR_SHAPE      # E > d/D
    assert etr.validate(hz.make_cfg(gw.scaled(w, T=0))) == etr.ERR_ARG
    assert etr.validate(hz.make_cfg(w, gemm_impl=etr.GEMM_TCGEN05)) == etr.ERR_UNSUPPORTED
    assert etr.lib().etr_validate(None) == etr.ERR_ARG
    x = torch.zeros(w.T, w.d, device="cuda")
    buf = etr.LayerBuffers(good)
    with pytest.raises(etr.EtrError) as e:
        etr.dispatch(good, None, buf.route, buf.Xp)
    assert e.value.code == etr.ERR_ARG
    with pytest.raises(etr.EtrError) as e:
        etr.dispatch(good, x.data_ptr() + 4, buf.route, buf.Xp)
    assert e.value.code == etr.ERR_ALIGN
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    out = etr.Buffers()
    base = (small.data_ptr() + 255) // 256 * 256
    assert etr.lib().etr_buffers_bind(C.byref(good), 0, C.c_void_p(base), C.c_size_t(512),
                                      C.byref(out)) == etr.ERR_WORKSPACE
    assert etr.launch_count() == n0
    torch.cuda.synchronize()
