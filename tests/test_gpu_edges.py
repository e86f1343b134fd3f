"""Edge cases of the CUDA path against the oracle: experts that receive no token, Top-1
routing (the paper's efficiency runs), k = E, capacity 1, a handful of tokens, group
sizes that take the generic pooling path, and tokens with more rows than the gather kernels stage."""
import numpy as np
import pytest
import torch

from gen import workloads as gw
from oracle import binding as ob
from tests import harness as hz

pytestmark = pytest.mark.gpu
etr = hz.etr
W = gw.WORKLOADS


def layer_vs_oracle(w, inp, mode, impl=etr.GEMM_AUTO):
    o = ob.Oracle("f32")
    fw = o.forward(inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], D=w.D, k=w.k,
                   capacity=w.capacity, mode=mode)
    bw = o.backward(fw, inp["X"], inp["R"], inp["W1g"], inp["W1u"], inp["W2"], inp["dY"])
    cfg = hz.make_cfg(w, mode=mode, gemm_impl=impl)
    dev = hz.upload(w, inp)
    buf = etr.LayerBuffers(cfg)
    out = dict(Y=torch.empty_like(dev.X), dX=torch.empty_like(dev.X), dR=torch.empty_like(dev.R),
               dW1g=torch.full_like(dev.W1g, float("nan")), dW1u=torch.full_like(dev.W1u, float("nan")),
               dW2=torch.full_like(dev.W2, float("nan")))
    etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, out["Y"])
    etr.layer_backward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, dev.dY, buf, out["dX"], out["dR"],
                       out["dW1g"], out["dW1u"], out["dW2"])
    torch.cuda.synchronize()
    assert buf.read_stats().error_word == 0
    got = hz.route_from_buffers(buf, cfg)
    hz.check_route_structure(hz.to_np(buf.delta), got, mode)
    identical = hz.assert_routes_match(fw.delta, fw.route, got, mode)
    assert identical, "these cases are built with clear margins"
    tol = 2e-2 if w.dtype == "bf16" else 1e-4
    for nm, ref, chain in (("Y", fw.Y, 4), ("dX", bw.dX, 6), ("dR", bw.dR, 4), ("dW1g", bw.dW1g, 6),
                           ("dW1u", bw.dW1u, 6), ("dW2", bw.dW2, 4)):
        hz.assert_close_rms(hz.to_np(out[nm]), ref, tol, nm, chain=chain)
    return fw, got, out


TC_FORMS = [etr.GEMM_TCGEN05, etr.GEMM_TCGEN05_2CTA, etr.GEMM_TCGEN05_2CTA_WIDE]


@pytest.mark.parametrize("dtype,impl", [("f32", etr.GEMM_AUTO), ("bf16", etr.GEMM_AUTO), ("bf16", etr.GEMM_SIMT)]
                         + [("bf16", f) for f in TC_FORMS])
def test_experts_without_tokens_get_zero_gradients(dtype, impl):
    """Token choice with every token pushed away from experts 2 and 5: their buffers stay
    empty, their weight gradients must be exactly zero, everything else must match."""
    w = gw.scaled(W["small"], T=384, d=256, D=8, E=8, h=128, dtype=dtype)
    inp = gw.make_inputs(w)
    lean = np.repeat(inp["R"], w.D, axis=1)              # expert directions in R^d
    X = inp["X"] - 0.5 * (lean[2] + lean[5])[None, :] * np.sqrt(w.d / w.D)
    inp["X"] = gw.round_to_bf16(X) if dtype == "bf16" else X.astype(np.float32)
    fw, got, out = layer_vs_oracle(w, inp, ob.MODE_TCR, impl)
    assert got.counts[2] == 0 and got.counts[5] == 0 and got.counts.sum() > 0
    for nm in ("dW1g", "dW1u", "dW2"):
        g = out[nm]
        assert bool((g[2] == 0).all()) and bool((g[5] == 0).all()), nm
    assert bool((out["dR"][2] == 0).all())


@pytest.mark.parametrize("impl", [etr.GEMM_AUTO] + TC_FORMS)
@pytest.mark.parametrize("k", [1, 8])
def test_top1_and_top_all(k, impl):
    """h = 192 and d = 256 leave ragged column tiles in every tile form."""
    w = gw.scaled(W["small"], T=300, d=256, D=8, E=8, h=192, k=k, cf=0.8)
    layer_vs_oracle(w, gw.make_inputs(w), ob.MODE_TCR, impl)


@pytest.mark.parametrize("impl", [etr.GEMM_AUTO] + TC_FORMS)
@pytest.mark.parametrize("mode", [ob.MODE_TCR, ob.MODE_ECR])
def test_capacity_one_and_few_tokens(mode, impl):
    w = gw.scaled(W["small"], T=5, d=128, D=8, E=4, h=64, cf=0.2)
    assert w.capacity == 1
    layer_vs_oracle(w, gw.make_inputs(w), mode, impl)


@pytest.mark.parametrize("impl", TC_FORMS)
def test_wide_columns_with_a_ragged_second_half(impl):
    """d = 640 and h = 320: the 512-column tiles of the wide form end in a partial second half
    (640 = 512 + 128) or have none at all (320), with 700 tokens per expert at most (ragged rows)."""
    w = gw.scaled(W["small"], T=1400, d=640, D=8, E=4, h=320, cf=1.0)
    layer_vs_oracle(w, gw.make_inputs(w), ob.MODE_ECR, impl)


@pytest.mark.parametrize("D,dtype", [(1, "f32"), (2, "bf16"), (4, "bf16"), (32, "bf16"), (24, "f32")])
def test_group_sizes(D, dtype):
    """D = 1 (plain cosine routing), sub-vector groups, wide groups and a group size that is
    neither a divisor nor a multiple of 8."""
    d = 768 if D == 24 else 512
    w = gw.scaled(W["small"], T=200, d=d, D=D, E=8, h=64, dtype=dtype)
    layer_vs_oracle(w, gw.make_inputs(w), ob.MODE_TCR)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_tokens_kept_by_every_expert_overflow_the_staged_row_lists(dtype):
    """Expert choice with C = T and 128 experts: every token has 128 rows, so the chunks of 8
    (combine) and 16 (fused dX) consecutive tokens hold 1024 and 2048 row entries, more than the
    512 those kernels stage in shared memory: the entries beyond are read in place.  T = 40 also
    leaves a ragged last chunk in both."""
    w = gw.scaled(W["small"], T=40, d=1024, D=8, E=128, h=64, cf=64.0, dtype=dtype)
    assert w.capacity == w.T
    fw, got, out = layer_vs_oracle(w, gw.make_inputs(w), ob.MODE_ECR)
    assert np.all(np.diff(got.tok_ptr) == w.E)


@pytest.mark.parametrize("d,D,dtype", [(2048, 16, "bf16"), (2048, 4, "bf16"), (2048, 8, "f32"), (4096, 32, "bf16"),
                                       (8192, 64, "bf16")])
def test_fused_dx_at_wide_hidden_sizes(d, D, dtype):
    """Hidden sizes of 2048, 4096 and 8192 in the fused dX kernel (whole 4 to 16 KiB rows per token and
    row of dXp), power-of-two and generic group sizes, a ragged last chunk of tokens (T = 215 =
    13 * 16 + 7), and expert choice with C = T / 4, which gives tokens anything from no row (zeros,
    X not read) to the rows of most of the 16 experts, so that one chunk's flat list of row entries
    crosses many token boundaries."""
    w = gw.scaled(W["small"], T=215, d=d, D=D, E=16, h=64, cf=2.0, dtype=dtype)
    fw, got, out = layer_vs_oracle(w, gw.make_inputs(w), ob.MODE_ECR)
    n = np.diff(got.tok_ptr)
    assert n.min() == 0 and n.max() >= 6 and n.sum() > 3 * w.T


def _affinity_on_device(w, inp, rows=None):
    cfg = hz.make_cfg(w if rows is None else gw.scaled(w, T=rows.stop - rows.start))
    X = hz.to_dev(inp["X"] if rows is None else inp["X"][rows], w)
    R = torch.from_numpy(inp["R"]).cuda()
    T, m = X.shape[0], w.d // w.D
    delta = torch.empty(T, w.E, dtype=torch.float32, device="cuda")
    Z = torch.empty(T, m, dtype=torch.float32, device="cuda")
    xnorm = torch.empty(T, dtype=torch.float32, device="cuda")
    rnorm = torch.empty(w.E, dtype=torch.float32, device="cuda")
    stats = torch.zeros(16, dtype=torch.int32, device="cuda")
    etr.affinity(cfg, X, R, delta, Z, xnorm, rnorm, stats)
    torch.cuda.synchronize()
    assert int(stats[6].item()) == 0            # error_word
    return delta, rnorm, stats


@pytest.mark.parametrize("T,d,D,E,dtype", [(1000, 256, 8, 7, "bf16"), (130, 512, 4, 64, "f32"), (4097, 2048, 8, 33, "bf16"),
                                            (127, 64, 2, 1, "bf16"), (20000, 1024, 4, 12, "bf16")])
def test_affinity_scores_on_the_tensor_cores(T, d, D, E, dtype):
    """Shapes the tensor-core score kernel takes (E <= 64, 32 | d/D): expert counts that are not a multiple of 4
    (scalar stores), a single expert, one K block, a ragged last tile of tokens, more tiles than SMs.  Affinities
    within the usual 1e-5, the batch maximum equal to the largest affinity stored, and a token's affinities the
    same bits whether it is scored in the whole batch or in a slice of it."""
    w = gw.scaled(W["small"], T=T, d=d, D=D, E=E, k=1, h=64, dtype=dtype)
    assert E <= 64 and (d // D) % 32 == 0
    inp = gw.make_inputs(w, weights=False)
    delta_ref, _, rnorm_ref, _ = ob.Oracle("f32").affinity(inp["X"], inp["R"], w.D)
    delta, rnorm, stats = _affinity_on_device(w, inp)
    got = hz.to_np(delta)
    hz.assert_affinity_close(got, delta_ref)
    assert np.allclose(hz.to_np(rnorm), rnorm_ref, rtol=1e-6, atol=0)
    u = int(np.float32(got.max()).view(np.uint32))
    key = (~u & 0xffffffff) if (u & 0x80000000) else (u | 0x80000000)
    assert int(stats[5].item()) & 0xffffffff == key
    rows = slice(T // 3, T // 3 + min(300, T - T // 3))
    part, _, _ = _affinity_on_device(w, inp, rows)
    assert torch.equal(part, delta[rows])


@pytest.mark.parametrize("E,dtype,d", [(16, "bf16", 640), (32, "f32", 640), (64, "bf16", 640), (64, "bf16", 512)])
def test_affinity_with_a_score_tile_for_every_sm(E, dtype, d):
    """38100 tokens: at least one 256-token tile per SM and a ragged last tile.  With d/D = 80 (16 divides it, 32
    does not) the fp32 score kernel takes its register-tiled form (2, 4 or 8 experts per lane for E <= 16, 32,
    64); with d/D = 64 the tensor-core kernel takes the same batch."""
    w = gw.scaled(W["small"], T=38100, d=d, D=8, E=E, h=64, dtype=dtype)
    inp = gw.make_inputs(w, weights=False)
    delta_ref, *_ = ob.Oracle("f32").affinity(inp["X"], inp["R"], w.D)
    cfg = hz.make_cfg(w)
    X = hz.to_dev(inp["X"], w)
    R = torch.from_numpy(inp["R"]).cuda()
    T, m = w.T, w.d // w.D
    delta = torch.empty(T, E, dtype=torch.float32, device="cuda")
    Z = torch.empty(T, m, dtype=torch.float32, device="cuda")
    xnorm = torch.empty(T, dtype=torch.float32, device="cuda")
    rnorm = torch.empty(E, dtype=torch.float32, device="cuda")
    stats = torch.zeros(16, dtype=torch.int32, device="cuda")
    etr.affinity(cfg, X, R, delta, Z, xnorm, rnorm, stats)
    torch.cuda.synchronize()
    got = hz.to_np(delta)
    hz.assert_affinity_close(got, delta_ref)
    u = int(np.float32(got.max()).view(np.uint32))
    key = (~u & 0xffffffff) if (u & 0x80000000) else (u | 0x80000000)
    assert int(stats[5].item()) & 0xffffffff == key


def test_sweep_modes_follow_the_step():
    """ETR_MODE_AUTO picks token choice before switch_step and expert choice from it on."""
    for step, want in ((999, etr.MODE_TCR), (1000, etr.MODE_ECR)):
        w = gw.scaled(W["sweep"], T=256, d=256, D=16, E=8, h=64, n_clusters=8, step=step)
        inp = gw.make_inputs(w)
        cfg = etr.make_config(T=w.T, d=w.d, D=w.D, E=w.E, k=w.k, h=w.h, capacity=w.capacity,
                              dtype=etr.BF16, mode=etr.MODE_AUTO, step=step, switch_step=w.switch_step,
                              adaptive=True)
        dev = hz.upload(w, inp)
        buf = etr.LayerBuffers(cfg)
        Y = torch.empty_like(dev.X)
        etr.layer_forward(cfg, dev.X, dev.R, dev.W1g, dev.W1u, dev.W2, buf, Y)
        st = buf.read_stats()
        assert st.mode == want and 1 <= st.C <= w.capacity
        o = ob.Oracle("f32")
        delta, *_ = o.affinity(inp["X"], inp["R"], w.D)
        assert st.C == ob.capacity_bound(w.d, w.E, w.capacity, 1, True, st.delta_max)
        if want == etr.MODE_ECR:
            assert np.all(hz.to_np(buf.counts) == min(st.C, w.T))
