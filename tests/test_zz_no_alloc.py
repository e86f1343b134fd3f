"""etr_select_static: the selection for callers that cannot allocate device memory.

Some users of the library (plugins inside a process whose device memory is owned by a
pool, code inside regions where cudaMalloc is forbidden because it synchronises the device)
cannot provide the scratch block etr_select wants.  etr_select_static keeps that scratch in
a fixed array inside the library instead.  This test calls it through the C ABI twice in a
row (the array keeps the previous call's contents, so the second call proves nothing stale
leaks through) and checks every routing output against etr_select bit for bit: the maps
are integers, so the tolerance is zero.  It lives in a file collected last so that a run
stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from gen import workloads as gw
from paper_2406_00023_b200 import etr

pytestmark = pytest.mark.gpu


def _routes(buf, cfg):
    st = buf.read_stats()
    n = st.rows_total
    return dict(topk=buf.topk_idx.cpu().numpy().copy(), counts=buf.counts.cpu().numpy().copy(),
                slot=buf.slot_token.cpu().numpy().copy(), gate=buf.gate.cpu().numpy().copy(),
                ptr=buf.tok_ptr.cpu().numpy().copy(), row=buf.tok_row.cpu().numpy()[:n].copy(),
                scalars=(st.mode, st.C, st.dropped, st.unrouted, st.rows_total))


def _affinities(w, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return (torch.randn(w.T, w.E, generator=g, device="cuda") / np.sqrt(w.d)).contiguous()


# T = 3000: one CTA per expert; T = 12000: each expert's keys split over a cluster of four CTAs;
# T = 65536 with E = 64 fills the fixed array to its last entry (the largest problem accepted).
SHAPES = [dict(T=3000), dict(T=12000), dict(T=65536, E=64, d=4096, D=16)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: f"T{s['T']}")
@pytest.mark.parametrize("mode", [etr.MODE_TCR, etr.MODE_ECR])
def test_select_static_matches_select_on_two_calls_in_a_row(mode, shape):
    w = gw.scaled(gw.WORKLOADS["small"], **shape)
    assert w.T * w.E <= etr.SELECT_STATIC_MAX_ENTRIES
    cfg = etr.make_config(T=w.T, d=w.d, D=w.D, E=w.E, k=w.k, h=w.h, capacity=w.capacity,
                          dtype=etr.BF16, mode=mode)
    ws = torch.empty(etr.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    for call in range(2):
        delta = _affinities(w, 1234 + call)          # different affinities on the second call
        ref_buf, got_buf = etr.LayerBuffers(cfg), etr.LayerBuffers(cfg)
        for b in (ref_buf, got_buf):
            b.stats.zero_()
            b.delta.copy_(delta)
        etr.select(cfg, ref_buf.delta, ref_buf.c.stats, ref_buf.route, ws)
        etr.select_static(cfg, got_buf.delta, got_buf.c.stats, got_buf.route)
        torch.cuda.synchronize()
        ref, got = _routes(ref_buf, cfg), _routes(got_buf, cfg)
        assert ref["scalars"][4] > 0
        for key in ref:
            if key == "scalars":
                assert ref[key] == got[key], (call, key)
            else:
                assert np.array_equal(ref[key], got[key]), (call, key)


def test_select_static_rejects_problems_beyond_its_fixed_scratch():
    too_big = etr.make_config(T=etr.SELECT_STATIC_MAX_ENTRIES // 64 + 64, d=4096, D=16, E=64, k=2,
                              h=2048, capacity=2048, dtype=etr.BF16, mode=etr.MODE_ECR)
    assert etr.validate(too_big) == etr.OK
    n0 = etr.launch_count()
    dummy = torch.zeros(64, device="cuda")
    route = etr.Route(*[dummy.data_ptr()] * 6)
    with pytest.raises(etr.EtrError) as e:
        etr.select_static(too_big, dummy, dummy, route)
    assert e.value.code == etr.ERR_WORKSPACE
    assert etr.launch_count() == n0
    # the same argument rules as etr_select: a route pointer off its 16-byte alignment is refused
    ok = etr.make_config(T=3000, d=1024, D=8, E=16, k=2, h=2816, capacity=469, dtype=etr.BF16, mode=etr.MODE_ECR)
    bad_route = etr.Route(*([dummy.data_ptr()] * 5 + [dummy.data_ptr() + 4]))
    with pytest.raises(etr.EtrError) as e:
        etr.select_static(ok, dummy, dummy, bad_route)
    assert e.value.code == etr.ERR_ALIGN
    assert etr.launch_count() == n0
