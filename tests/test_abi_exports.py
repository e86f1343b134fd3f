"""The C-ABI library builds without a GPU, loads, and exports every function include/etr.h
declares; host-side argument checks work with no device present."""
import ctypes
import os
import re

from paper_2406_00023_b200 import build as etr_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "etr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(etr_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(etr_build.build())
    names = declared_functions()
    assert len(names) >= 23
    for n in names:
        assert hasattr(lib, n), f"{n} declared in etr.h but not exported"


def test_binding_lists_the_same_entry_points():
    from paper_2406_00023_b200 import etr
    assert sorted(etr.EXPORTS) == declared_functions()


def test_host_side_validation_needs_no_gpu():
    from paper_2406_00023_b200 import etr
    good = etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=160, dtype=etr.F32)
    assert etr.validate(good) == etr.OK
    assert etr.c_stride(good) == 256
    assert etr.workspace_bytes(good) > 0
    assert etr.validate(etr.make_config(T=512, d=256, D=3, E=8, k=2, h=512, capacity=160, dtype=etr.F32)) == etr.ERR_SHAPE
    assert etr.validate(etr.make_config(T=512, d=256, D=4, E=8, k=9, h=512, capacity=160, dtype=etr.F32)) == etr.ERR_SHAPE
    assert etr.validate(etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=0, dtype=etr.F32)) == etr.ERR_ARG
    assert etr.validate(etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=160, dtype=5)) == etr.ERR_ARG
    assert "aligned" in etr.status_string(etr.ERR_ALIGN)
    n = ctypes.c_size_t(0)
    assert etr.lib().etr_buffers_bytes(ctypes.byref(good), 1, ctypes.byref(n)) == etr.OK and n.value > 1 << 20
    # struct layouts the binding relies on
    assert ctypes.sizeof(etr.Config) == 112 and ctypes.sizeof(etr.Stats) == 64
    # fp32 master weights under bf16 activations are taken (rounded to bf16 in the tail of the workspace, which
    # grows by three weight tensors of 2 bytes); bf16 weights under fp32 activations have no kernel
    assert etr.validate(etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=160, dtype=etr.F32,
                                        weight_dtype=etr.BF16)) == etr.ERR_UNSUPPORTED
    b16 = etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=160, dtype=etr.BF16)
    mixed = etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=160, dtype=etr.BF16, weight_dtype=etr.F32)
    assert etr.validate(mixed) == etr.OK
    assert etr.workspace_bytes(mixed) == etr.workspace_bytes(b16) + 3 * 2 * 8 * 256 * 512


def test_layout_gives_the_offsets_bind_uses():
    from paper_2406_00023_b200 import etr
    for staging, gate in ((0, etr.GATE_AFFINITY), (1, etr.GATE_SOFTMAX)):
        cfg = etr.make_config(T=512, d=256, D=4, E=8, k=2, h=512, capacity=160, dtype=etr.BF16, gate_mode=gate)
        lay = etr.layout(cfg, bool(staging))
        n = ctypes.c_size_t(0)
        assert etr.lib().etr_buffers_bytes(ctypes.byref(cfg), staging, ctypes.byref(n)) == etr.OK
        assert lay.total_bytes == n.value and lay.C_stride == 256 and lay.ws_bytes == etr.workspace_bytes(cfg)
        base = 1 << 20                                   # binding only computes addresses: no memory is touched
        b = etr.Buffers()
        assert etr.lib().etr_buffers_bind(ctypes.byref(cfg), staging, ctypes.c_void_p(base),
                                          ctypes.c_size_t(n.value), ctypes.byref(b)) == etr.OK
        for name in ("delta", "Z", "xnorm", "rnorm", "Xp", "G", "U", "H", "O", "dO", "dG", "dU", "dXp", "dgate", "ws"):
            assert getattr(b, name) == base + getattr(lay, name), name
            assert getattr(lay, name) % 256 == 0
        assert b.route.slot_token == base + lay.slot_token and b.route.tok_row == base + lay.tok_row
        assert b.stats == base + lay.stats
        if staging:
            assert b.X_dev == base + lay.X_dev and b.lse == base + lay.lse and lay.ddelta > lay.lse > 0
        else:
            assert lay.X_dev == 0 and lay.lse == 0 and not b.X_dev
