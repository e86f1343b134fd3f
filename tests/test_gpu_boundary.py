"""Behaviour the C ABI promises besides the numbers of the default path: fp32 weight gradients
(grad_fp32), a selection that may be repeated on one stats block, the bounded device-side wait,
whose expiry must surface as ETR_ERR_TIMEOUT and leave the stream usable, and the selection cut by
a threshold on the sum of affinity scores (bit-exact against the oracle's select_thresholded)."""
import numpy as np
import pytest
import torch

from gen import workloads as gw
from oracle import binding as ob
from tests import harness as hz
from tests.test_gpu_parity import case, override_of, run_select, routes_equal

pytestmark = pytest.mark.gpu
etr = hz.etr

TC_FORMS = [etr.GEMM_AUTO, etr.GEMM_SIMT, etr.GEMM_TCGEN05, etr.GEMM_TCGEN05_2CTA, etr.GEMM_TCGEN05_2CTA_WIDE]


@pytest.mark.parametrize("impl", TC_FORMS)
@pytest.mark.parametrize("name", ["small_s", "mid_s", "sweep_s_ecr"])
def test_fp32_weight_gradients(name, impl):
    """grad_fp32: the three weight gradients leave the accumulators as fp32.  Fed with the
    oracle's stage inputs on the bf16 grid, what is left is the summation order (fp32 against
    double) and, for dW1, the kernel's own bf16 store of dG and dU in between; rounded to bf16 they
    must reproduce the bf16 outputs of the default path bit for bit."""
    w, inp, o, fw, bw = case(name)
    dev = hz.upload(w, inp)
    grid = gw.round_to_bf16
    dOq, Gq, Uq, Hq = grid(bw.dO), grid(fw.G), grid(fw.U), grid(fw.H)
    ref = o.expert_ffn_bwd(dOq, fw.Xp, Gq, Uq, Hq, fw.route, inp["W1g"], inp["W1u"], inp["W2"])
    outs = {}
    for g32 in (False, True):
        cfg = hz.make_cfg(w, gemm_impl=impl, grad_fp32=g32)
        buf = etr.LayerBuffers(cfg)
        hz.upload_route(buf, fw.route)
        buf.stats.zero_()
        etr.dispatch(cfg, dev.X, buf.route, buf.Xp)
        for nm, a in (("dO", dOq), ("G", Gq), ("U", Uq), ("H", Hq)):
            getattr(buf, nm).copy_(hz.to_dev(a, w))
        dt = torch.float32 if g32 else torch.bfloat16
        dW = [torch.full(t.shape, float("nan"), dtype=dt, device="cuda") for t in (dev.W1g, dev.W1u, dev.W2)]
        ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        etr.expert_ffn_bwd(cfg, buf.route, buf.dO, buf.Xp, buf.G, buf.U, buf.H, dev.W1g, dev.W1u, dev.W2,
                           buf.dG, buf.dU, buf.dXp, dW[0], dW[1], dW[2], buf.c.stats, ws)
        assert buf.read_stats().error_word == 0
        outs[g32] = dW
    for j, nm in enumerate(("dW1g", "dW1u", "dW2")):
        got32 = outs[True][j]
        assert got32.dtype == torch.float32 and not bool(torch.isnan(got32).any())
        assert torch.equal(got32.to(torch.bfloat16), outs[False][j]), f"{nm}: bf16(fp32 output) != bf16 output"
    # dW2 = dO^T H from inputs on the grid: only the summation order is left
    hz.assert_within(hz.to_np(outs[True][2]), ref[5], 2e-5, "dW2 fp32")
    # dW1 = dG^T Xp with the kernel's stored (bf16) dG, dU: one store on the path
    hz.assert_close_rms(hz.to_np(outs[True][0]), ref[3], 2e-2, "dW1g fp32", chain=1)
    hz.assert_close_rms(hz.to_np(outs[True][1]), ref[4], 2e-2, "dW1u fp32", chain=1)


def test_layer_with_fp32_weight_gradients():
    """Whole layer with grad_fp32: the weight gradients lose their final rounding; everything
    else is bit-identical to the default layer."""
    w, inp, o, fw, bw = case("small_s")
    dev = hz.upload(w, inp)
    res = {}
    for g32 in (False, True):
        cfg = hz.make_cfg(w, grad_fp32=g32)
        buf = etr.LayerBuffers(cfg)
        dt = torch.float32 if g32 else torch.bfloat16
        out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
                   dW1g=torch.empty(dev.W1g.shape, dtype=dt, device="cuda"),
                   dW1u=torch.empty(dev.W1u.shape, dtype=dt, device="cuda"),
                   dW2=torch.empty(dev.W2.shape, dtype=dt, device="cuda"))
        etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
        etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                           out["dW1g"], out["dW1u"], out["dW2"])
        torch.cuda.synchronize()
        assert buf.read_stats().error_word == 0
        res[g32] = out
    for k in ("Y", "dX", "dR"):
        assert torch.equal(res[False][k], res[True][k]), k
    for k, chain in (("dW1g", 5), ("dW1u", 5), ("dW2", 3)):
        assert torch.equal(res[True][k].to(torch.bfloat16), res[False][k]), k
        hz.assert_close_rms(hz.to_np(res[True][k]), getattr(bw, k), 2e-2, k + " fp32", chain=chain)


@pytest.mark.parametrize("impl", [etr.GEMM_AUTO, etr.GEMM_TCGEN05, etr.GEMM_SIMT])
def test_fp32_master_weights_with_bf16_activations(impl):
    """weight_dtype = fp32 under dtype = bf16: the library rounds the weights to bf16 (nearest even) for the
    GEMMs and returns fp32 weight gradients.  Every output must equal, bit for bit, the bf16 layer with
    grad_fp32 run on weights rounded the same way beforehand; the fp32 weights here are not on the bf16 grid."""
    w, inp, o, fw, bw = case("small_s")
    dev = hz.upload(w, inp)
    g = torch.Generator(device="cuda").manual_seed(7)
    master = {}
    for k in ("W1g", "W1u", "W2"):
        wb = getattr(dev, k)
        # the same values to bf16 precision, plus bits below it that rounding must remove again
        noise = (torch.rand(wb.shape, device="cuda", generator=g) - 0.5) * 2.0 ** -10
        m32 = wb.float() * (1.0 + noise)
        assert torch.equal(m32.to(torch.bfloat16), wb) and not torch.equal(m32, wb.float())
        master[k] = m32.contiguous()
    res = {}
    for mixed in (False, True):
        cfg = hz.make_cfg(w, gemm_impl=impl, grad_fp32=not mixed,
                          **(dict(weight_dtype=etr.F32) if mixed else {}))
        W = [master[k] if mixed else getattr(dev, k) for k in ("W1g", "W1u", "W2")]
        buf = etr.LayerBuffers(cfg)
        out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
                   dW1g=torch.empty(dev.W1g.shape, dtype=torch.float32, device="cuda"),
                   dW1u=torch.empty(dev.W1u.shape, dtype=torch.float32, device="cuda"),
                   dW2=torch.empty(dev.W2.shape, dtype=torch.float32, device="cuda"))
        etr.layer_forward(cfg, dev.X, dev.R, *W, buf, out["Y"])
        etr.layer_backward(cfg, dev.X, dev.R, *W, dev.dY, buf, out["dX"], out["dR"], out["dW1g"], out["dW1u"],
                           out["dW2"])
        torch.cuda.synchronize()
        assert buf.read_stats().error_word == 0
        # the stage calls round the weights themselves: same G, U, H, O and gradients as the layer's
        st = dict(G=torch.empty_like(buf.G), U=torch.empty_like(buf.U), H=torch.empty_like(buf.H),
                  O=torch.empty_like(buf.O), dG=torch.empty_like(buf.dG), dU=torch.empty_like(buf.dU),
                  dXp=torch.empty_like(buf.dXp), dW1g=torch.empty_like(out["dW1g"]),
                  dW1u=torch.empty_like(out["dW1u"]), dW2=torch.empty_like(out["dW2"]))
        ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        etr.expert_ffn(cfg, buf.route, buf.Xp, *W, st["G"], st["U"], st["H"], st["O"], buf.c.stats, ws)
        etr.expert_ffn_bwd(cfg, buf.route, buf.dO, buf.Xp, buf.G, buf.U, buf.H, *W, st["dG"], st["dU"], st["dXp"],
                           st["dW1g"], st["dW1u"], st["dW2"], buf.c.stats, ws)
        torch.cuda.synchronize()
        live = buf.slot_token >= 0                   # rows beyond an expert's count are not part of the result
        for k in ("G", "U", "H", "O", "dG", "dU", "dXp"):
            assert torch.equal(st[k].view(live.numel(), -1)[live], getattr(buf, k).view(live.numel(), -1)[live]), k
        for k in ("dW1g", "dW1u", "dW2"):
            assert torch.equal(st[k], out[k]), k
        res[mixed] = out
    for k in res[False]:
        assert torch.equal(res[False][k], res[True][k]), k
    hz.assert_close_rms(hz.to_np(res[True]["dW2"]), bw.dW2, 2e-2, "dW2 fp32 master", chain=3)


def test_mixed_weight_dtype_is_bf16_activations_only():
    w = gw.WORKLOADS["tiny"]
    assert w.dtype == "f32"
    with pytest.raises(etr.EtrError):
        etr.workspace_bytes(hz.make_cfg(w, weight_dtype=etr.BF16))      # fp32 activations, bf16 weights


@pytest.mark.parametrize("name", ["small_s", "sweep_s_ecr"])
def test_select_may_be_repeated_on_one_stats_block(name):
    """The selection sets every counter it reports: a second selection on the same stats (another
    step or capacity of a sweep, with delta_max_key left in place by etr_affinity) must give what
    a selection on fresh stats gives."""
    w, inp, o, fw, _ = case(name)
    ov = override_of(name)
    cfg = hz.make_cfg(w, delta_max_override=ov)
    buf, first = run_select(w, cfg, fw.delta)
    assert routes_equal(fw.route, first)
    ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    # again, and then once more with the other mode and a smaller capacity, never clearing stats
    etr.select(cfg, buf.delta, buf.c.stats, buf.route, ws)
    assert routes_equal(fw.route, hz.route_from_buffers(buf, cfg))
    other = ob.MODE_ECR if hz.mode_of(w) == ob.MODE_TCR else ob.MODE_TCR
    w2 = gw.scaled(w, cf=w.cf / 2, adaptive=False)
    cfg2 = hz.make_cfg(w2, mode=other)
    buf2 = etr.LayerBuffers(cfg2)
    buf2.delta.copy_(buf.delta)
    buf2.stats.copy_(buf.stats)                   # carries the first selection's counters
    etr.select(cfg2, buf2.delta, buf2.c.stats, buf2.route, ws)
    ref2 = o.select(fw.delta, w.k, other, w2.capacity, w2.C_stride)
    assert routes_equal(ref2, hz.route_from_buffers(buf2, cfg2))
    etr.select_static(cfg2, buf2.delta, buf2.c.stats, buf2.route)
    assert routes_equal(ref2, hz.route_from_buffers(buf2, cfg2))


def test_bounded_wait_expires_as_a_status_and_the_stream_stays_usable():
    """The failure path of the GEMM pipeline without a failure: a one-warp kernel waits, with the
    pipeline's wait routine and a limit of 1e5 cycles (about 50 microseconds), on a barrier nothing
    arrives on.  The kernel must return by itself, etr_read_stats must report ETR_ERR_TIMEOUT, and
    an ordinary layer call on the same stream and buffers must then pass as usual."""
    w, inp, o, fw, bw = case("small_s")
    cfg = hz.make_cfg(w)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    buf.stats.zero_()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    etr.selftest_bounded_wait(buf.c.stats, 100_000)
    t1.record()
    with pytest.raises(etr.EtrError) as e:
        buf.read_stats()
    assert e.value.code == etr.ERR_TIMEOUT
    assert int(buf.stats[6].item()) == 0x7c08
    assert t0.elapsed_time(t1) < 50.0, "the wait did not end near its limit"
    with pytest.raises(etr.EtrError) as e:
        etr.selftest_bounded_wait(buf.c.stats, 0)
    assert e.value.code == etr.ERR_ARG
    # the next ordinary call: same stream, same buffers; etr_layer_forward clears the stats
    Y = torch.empty_like(dev.X)
    etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, Y)
    st = buf.read_stats()
    assert st.error_word == 0
    hz.assert_close_rms(hz.to_np(Y), fw.Y, 2e-2, "Y after an expired wait", chain=4)
    # a limit passed through the config reaches the GEMM kernels; a generous one changes nothing
    cfg_l = hz.make_cfg(w, wait_limit_cycles=2_000_000_000)
    Y2 = torch.empty_like(dev.X)
    etr.layer_forward(cfg_l, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, Y2)
    assert buf.read_stats().error_word == 0 and torch.equal(Y, Y2)


THRESHOLD_CASES = [
    # (T, E, k, C, mode, flags, tau_expert, tau_token)
    (1000, 16, 2, 160, ob.MODE_TCR, 1, 2.0, np.inf),
    (1000, 16, 2, 160, ob.MODE_ECR, 1, 3.5, np.inf),
    (1000, 16, 4, 300, ob.MODE_TCR, 2, np.inf, 0.12),
    (1000, 16, 4, 300, ob.MODE_TCR, 3, 1.5, 0.12),
    (777, 8, 2, 64, ob.MODE_ECR, 1, 1e-3, np.inf),            # below the first score: one token each
    (777, 8, 2, 64, ob.MODE_ECR, 1, 0.0, np.inf),             # nothing kept
    (777, 8, 2, 64, ob.MODE_TCR, 3, np.inf, np.inf),          # no cut at all
    (12000, 32, 2, 900, ob.MODE_ECR, 1, 30.0, np.inf),        # expert's keys split over a cluster of CTAs
    (12000, 32, 2, 900, ob.MODE_TCR, 3, 12.0, 0.2),
]


@pytest.mark.parametrize("T,E,k,C,mode,flags,tau_e,tau_t", THRESHOLD_CASES)
def test_selection_with_a_threshold_on_the_affinity_sum(T, E, k, C, mode, flags, tau_e, tau_t):
    """etr_select with threshold_mode set against the oracle's select_thresholded on the same affinity
    bits: every map, count and counter identical (the sums are integers on both sides)."""
    w = gw.scaled(gw.WORKLOADS["small"], T=T, E=E, k=k, d=1024, D=8, cf=(C - 0.5) * E / (T * k))
    assert w.capacity == C
    rng = np.random.default_rng(T + 31 * flags)
    delta = (rng.standard_normal((T, E)) / 12).astype(np.float32)       # mixed signs, |delta| ~ 0.08
    delta[rng.random((T, E)) < 0.02] = np.float32(0.0625)               # and some exact ties
    o = ob.Oracle("f32")
    ref = o.select_thresholded(delta, k, mode, C, w.C_stride, flags, tau_e, tau_t)
    cfg = hz.make_cfg(w, mode=mode, threshold_mode=flags, threshold_tau=tau_e, threshold_tau_token=tau_t)
    _, got = run_select(w, cfg, delta)
    assert routes_equal(ref, got)
    if flags & 1 and np.isfinite(tau_e) and tau_e > 0.01:
        assert np.any(got.counts < min(C, T)), "the threshold was meant to bite"
    buf = etr.LayerBuffers(cfg)
    buf.stats.zero_()
    buf.delta.copy_(torch.from_numpy(delta))
    etr.select_static(cfg, buf.delta, buf.c.stats, buf.route)
    assert routes_equal(ref, hz.route_from_buffers(buf, cfg))


@pytest.mark.parametrize("mode,flags", [(ob.MODE_TCR, 3), (ob.MODE_ECR, 1)])
def test_layer_with_a_threshold_on_the_affinity_sum(mode, flags):
    """The whole layer with the threshold on: routing identical to the oracle's, outputs and
    gradients within the usual bounds (the stages after the selection do not know about it)."""
    w, inp, o, _, _ = case("small_s")
    tau_e, tau_t = 2.5, 0.09
    fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k, capacity=w.capacity,
                   mode=mode, threshold_mode=flags, tau_expert=tau_e, tau_token=tau_t)
    bw = o.backward(fw, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    assert 0 < fw.route.tok_ptr[-1] < o.select(fw.delta, w.k, mode, w.capacity, w.C_stride).tok_ptr[-1]
    cfg = hz.make_cfg(w, mode=mode, threshold_mode=flags, threshold_tau=tau_e, threshold_tau_token=tau_t)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
               dW1g=torch.empty_like(dev.W1g), dW1u=torch.empty_like(dev.W1u), dW2=torch.empty_like(dev.W2))
    etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
    etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                       out["dW1g"], out["dW1u"], out["dW2"])
    torch.cuda.synchronize()
    assert buf.read_stats().error_word == 0
    got = hz.route_from_buffers(buf, cfg)
    # the device's affinities differ from the oracle's in the last bits, and a running sum within
    # a few 2^-32 of tau may then stop one candidate earlier or later: compare on the oracle's route
    # only when the maps agree, which these seeds give
    assert hz.assert_routes_match(fw.delta, fw.route, got, mode), "threshold crossings have clear margins here"
    for nm, ref, chain in (("Y", fw.Y, 4), ("dX", bw.dX, 6), ("dR", bw.dR, 4), ("dW1g", bw.dW1g, 6),
                           ("dW1u", bw.dW1u, 6), ("dW2", bw.dW2, 4)):
        hz.assert_close_rms(hz.to_np(out[nm]), ref, 2e-2, nm, chain=chain)


@pytest.mark.parametrize("impl", [etr.GEMM_AUTO, etr.GEMM_TCGEN05, etr.GEMM_TCGEN05_2CTA, etr.GEMM_TCGEN05_2CTA_WIDE])
@pytest.mark.parametrize("name,cf", [("small_s", 1.25), ("sweep_s_tcr", 0.5)])
def test_top1_combine_in_the_down_gemm_epilogue(name, cf, impl):
    """Top-1 token choice: with the combine folded into the down GEMM's epilogue (the default there)
    the combine kernel does not run and every output equals the unfused path bit for bit, on all
    tile forms; tokens without a row (capacity factor 0.5 drops many) get exact zeros; with k = 2 the
    switch changes nothing."""
    w0, inp, o, _, _ = case(name)
    w = gw.scaled(w0, k=1, cf=cf, adaptive=False)
    dev = hz.upload(w, inp)
    res, names = {}, {}
    for fuse in (etr.FUSE_OFF, etr.FUSE_AUTO):
        cfg = hz.make_cfg(w, mode=ob.MODE_TCR, gemm_impl=impl, fuse_combine=fuse)
        buf = etr.LayerBuffers(cfg)
        out = dict(Y=torch.full_like(dev.X, float("nan")), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
                   dW1g=torch.empty_like(dev.W1g), dW1u=torch.empty_like(dev.W1u), dW2=torch.empty_like(dev.W2))
        etr.timing_enable(True)
        etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
        names[fuse] = [n for n, _ in etr.timing_collect()]
        etr.timing_enable(False)
        etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                           out["dW1g"], out["dW1u"], out["dW2"])
        torch.cuda.synchronize()
        st = buf.read_stats()
        assert st.error_word == 0
        out["O"] = buf.O.clone()
        res[fuse] = (out, st, hz.to_np(buf.tok_ptr))
    assert "combine_kernel" in names[etr.FUSE_OFF] and "combine_kernel" not in names[etr.FUSE_AUTO]
    assert "zero_unrouted_kernel" in names[etr.FUSE_AUTO]
    a, b = res[etr.FUSE_OFF][0], res[etr.FUSE_AUTO][0]
    for k in a:
        assert torch.equal(a[k], b[k]), k
    st, ptr = res[etr.FUSE_AUTO][1], res[etr.FUSE_AUTO][2]
    unrouted = np.diff(ptr) == 0
    assert st.unrouted == int(unrouted.sum())
    if cf < 1:
        assert st.unrouted > 0
    assert np.all(hz.to_np(b["Y"])[unrouted] == 0) and not np.isnan(hz.to_np(b["Y"])).any()
    # against the oracle as well
    fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=1, capacity=w.capacity,
                   mode=ob.MODE_TCR)
    hz.assert_close_rms(hz.to_np(b["Y"]), fw.Y, 2e-2, "Y (combine in the epilogue)", chain=4)
    # k = 2: a token's rows lie in different experts' tiles; the switch must leave the path alone
    w2 = gw.scaled(w0, adaptive=False)
    cfg2 = hz.make_cfg(w2, mode=ob.MODE_TCR, gemm_impl=impl, fuse_combine=etr.FUSE_ON)
    buf2 = etr.LayerBuffers(cfg2)
    Y2 = torch.empty_like(dev.X)
    etr.timing_enable(True)
    etr.layer_forward(cfg2, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf2, Y2)
    assert "combine_kernel" in [n for n, _ in etr.timing_collect()]
    etr.timing_enable(False)


@pytest.mark.parametrize("name", ["small_s", "sweep_s_ecr"])
def test_layer_calls_can_be_captured_in_a_cuda_graph(name):
    """etr_layer_forward + etr_layer_backward enqueue only stream work (kernels and one memset; mode,
    capacity and row counts stay on the device), so a step can be captured once and replayed: the
    replays must give the bits of the direct calls, also after the inputs changed in place."""
    w, inp, o, fw, bw = case(name)
    cfg = hz.make_cfg(w, delta_max_override=override_of(name) if w.adaptive else -1.0)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
               dW1g=torch.empty_like(dev.W1g), dW1u=torch.empty_like(dev.W1u), dW2=torch.empty_like(dev.W2))

    def step():
        etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
        etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                           out["dW1g"], out["dW1u"], out["dW2"])

    step()                                        # direct calls first (and every kernel's one-time set-up)
    torch.cuda.synchronize()
    ref = {k: v.clone() for k, v in out.items()}
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for v in out.values():
        v.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert buf.read_stats().error_word == 0
    for k in ref:
        assert torch.equal(out[k], ref[k]), k
    # other tokens in the same buffers: the replay follows the data (routing is decided on the device)
    X0 = dev.X.clone()
    dev.X.copy_(X0.flip(0))
    graph.replay()
    torch.cuda.synchronize()
    got = {k: v.clone() for k, v in out.items()}
    step()
    torch.cuda.synchronize()
    for k in got:
        assert torch.equal(out[k], got[k]), k
    assert not torch.equal(got["Y"], ref["Y"])
