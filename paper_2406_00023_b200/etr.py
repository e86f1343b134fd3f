"""ctypes binding of libetr (include/etr.h).  Argument marshalling only.

Tensors are torch CUDA tensors used as plain device memory; the current torch stream is
passed to every call.  The library is loaded from this package's directory and loading
fails loudly if it has not been built (python -m paper_2406_00023_b200.build).
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ETR_LIB_PATH") or os.path.join(_HERE, "libetr.so")   # override: another build of the library

OK, ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = range(8)
F32, BF16 = 0, 1
MODE_AUTO, MODE_TCR, MODE_ECR = 0, 1, 2
GEMM_AUTO, GEMM_SIMT, GEMM_TCGEN05, GEMM_TCGEN05_2CTA, GEMM_TCGEN05_2CTA_WIDE = 0, 1, 2, 3, 4
FUSE_AUTO, FUSE_OFF, FUSE_ON = 0, 1, 2
GATE_AFFINITY, GATE_SOFTMAX = 0, 1
THRESHOLD_OFF, THRESHOLD_EXPERT, THRESHOLD_TOKEN = 0, 1, 2

EXPORTS = [
    "etr_status_string", "etr_validate", "etr_c_stride", "etr_workspace_bytes", "etr_buffers_bytes",
    "etr_buffers_bind", "etr_layout", "etr_read_status", "etr_affinity", "etr_select", "etr_select_static", "etr_dispatch", "etr_expert_ffn", "etr_combine",
    "etr_combine_bwd", "etr_expert_ffn_bwd", "etr_dispatch_bwd", "etr_select_bwd", "etr_affinity_bwd",
    "etr_gate_softmax", "etr_gate_softmax_bwd", "etr_affinity_bwd_dense", "etr_load_stats",
    "etr_layer_forward", "etr_layer_backward", "etr_layer_step_host", "etr_layer_step_host_begin",
    "etr_layer_step_host_wait", "etr_read_stats", "etr_selftest_bounded_wait",
    "etr_launch_count", "etr_timing_enable", "etr_timing_collect",
]


class Config(C.Structure):
    _fields_ = [("T", C.c_int32), ("d", C.c_int32), ("D", C.c_int32), ("E", C.c_int32),
                ("k", C.c_int32), ("h", C.c_int32), ("capacity", C.c_int32), ("c_floor", C.c_int32),
                ("adaptive", C.c_int32), ("delta_max_override", C.c_float),
                ("step", C.c_int64), ("switch_step", C.c_int64), ("mode", C.c_int32),
                ("dtype", C.c_int32), ("gemm_impl", C.c_int32), ("fuse_dispatch", C.c_int32),
                ("gate_mode", C.c_int32), ("grad_fp32", C.c_int32), ("weight_dtype", C.c_int32),
                ("threshold_mode", C.c_int32), ("threshold_tau", C.c_float),
                ("threshold_tau_token", C.c_float), ("wait_limit_cycles", C.c_int64),
                ("fuse_combine", C.c_int32), ("reserved0", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("mode", C.c_int32), ("C", C.c_int32), ("dropped", C.c_int32),
                ("unrouted", C.c_int32), ("delta_max", C.c_float), ("delta_max_key", C.c_uint32),
                ("error_word", C.c_int32), ("rows_total", C.c_int32), ("reserved", C.c_int32 * 8)]


class Route(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("topk_idx", "counts", "slot_token", "gate", "tok_ptr", "tok_row")]


class Buffers(C.Structure):
    _fields_ = [("stats", C.c_void_p), ("route", Route)] + \
               [(n, C.c_void_p) for n in ("delta", "Z", "xnorm", "rnorm", "Xp", "G", "U", "H", "O",
                                          "dO", "dG", "dU", "dXp", "dgate", "ws")] + \
               [("ws_bytes", C.c_size_t)] + \
               [(n, C.c_void_p) for n in ("X_dev", "dY_dev", "Y_dev", "dX_dev", "lse", "ddelta")]


class LayoutInfo(C.Structure):
    _fields_ = [("C_stride", C.c_int32), ("reserved", C.c_int32)] + \
               [(n, C.c_size_t) for n in ("total_bytes", "ws_bytes", "stats", "topk_idx", "counts", "slot_token",
                                          "gate", "tok_ptr", "tok_row", "delta", "Z", "xnorm", "rnorm", "Xp", "G",
                                          "U", "H", "O", "dO", "dG", "dU", "dXp", "dgate", "ws", "X_dev", "dY_dev",
                                          "Y_dev", "dX_dev", "lse", "ddelta")]


class EtrError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (etr_status {code})")


_lib = None


def lib():
    """The loaded shared library.  Raises if it is missing: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not built; run `python -m paper_2406_00023_b200.build`")
        l = C.CDLL(LIB_PATH)
        l.etr_status_string.restype = C.c_char_p
        l.etr_status_string.argtypes = [C.c_int]
        l.etr_launch_count.restype = C.c_int64
        l.etr_c_stride.restype = C.c_int32
        _lib = l
    return _lib


def status_string(code: int) -> str:
    return lib().etr_status_string(int(code)).decode()


def launch_count() -> int:
    return int(lib().etr_launch_count())


def timing_enable(on: bool) -> None:
    lib().etr_timing_enable(int(bool(on)))


def timing_collect(max_records: int = 1 << 16):
    """[(kernel name, milliseconds)] for every launch since timing was enabled."""
    names = C.create_string_buffer(max_records * 48)
    ms = (C.c_float * max_records)()
    f = lib().etr_timing_collect
    f.restype = C.c_int64
    n = f(names, C.c_size_t(len(names)), ms, C.c_int64(max_records))
    return list(zip(names.value.decode().split("\n")[:n], [float(ms[i]) for i in range(n)]))


def _check(code, where):
    if code != OK:
        raise EtrError(code, where)


def _p(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(*, T, d, D, E, k, h, capacity, dtype, mode=MODE_AUTO, step=0, switch_step=0,
                adaptive=False, c_floor=1, delta_max_override=-1.0, gemm_impl=GEMM_AUTO,
                fuse_dispatch=0, gate_mode=0, grad_fp32=False, weight_dtype=None, threshold_mode=0,
                threshold_tau=float("inf"), threshold_tau_token=float("inf"), wait_limit_cycles=0,
                fuse_combine=0) -> Config:
    return Config(T=T, d=d, D=D, E=E, k=k, h=h, capacity=capacity, c_floor=c_floor,
                  adaptive=int(bool(adaptive)), delta_max_override=float(delta_max_override),
                  step=int(step), switch_step=int(switch_step), mode=int(mode), dtype=int(dtype),
                  gemm_impl=int(gemm_impl), fuse_dispatch=int(fuse_dispatch), gate_mode=int(gate_mode),
                  grad_fp32=int(bool(grad_fp32)), weight_dtype=int(dtype if weight_dtype is None else weight_dtype),
                  threshold_mode=int(threshold_mode), threshold_tau=float(threshold_tau),
                  threshold_tau_token=float(threshold_tau_token), wait_limit_cycles=int(wait_limit_cycles),
                  fuse_combine=int(fuse_combine), reserved0=0)


def torch_dtype(cfg: Config):
    return torch.bfloat16 if cfg.dtype == BF16 else torch.float32


def validate(cfg: Config) -> int:
    return lib().etr_validate(C.byref(cfg))


def c_stride(cfg: Config) -> int:
    return lib().etr_c_stride(C.byref(cfg))


def layout(cfg: Config, host_staging: bool = False) -> LayoutInfo:
    """Offsets of every buffer inside the block etr_buffers_bind carves."""
    out = LayoutInfo()
    _check(lib().etr_layout(C.byref(cfg), int(host_staging), C.byref(out)), "etr_layout")
    return out


def workspace_bytes(cfg: Config) -> int:
    n = C.c_size_t(0)
    _check(lib().etr_workspace_bytes(C.byref(cfg), C.byref(n)), "etr_workspace_bytes")
    return n.value


class LayerBuffers:
    """One device block carved by etr_buffers_bind, with typed tensor views of each member."""

    def __init__(self, cfg: Config, host_staging: bool = False, device="cuda"):
        n = C.c_size_t(0)
        _check(lib().etr_buffers_bytes(C.byref(cfg), int(host_staging), C.byref(n)), "etr_buffers_bytes")
        self.cfg = cfg
        self.nbytes = n.value
        self.block = torch.empty(n.value + 256, dtype=torch.uint8, device=device)
        base = (self.block.data_ptr() + 255) // 256 * 256
        self._base_off = base - self.block.data_ptr()
        self.c = Buffers()
        _check(lib().etr_buffers_bind(C.byref(cfg), int(host_staging), C.c_void_p(base),
                                      C.c_size_t(n.value), C.byref(self.c)), "etr_buffers_bind")
        T, E, d, h, k = cfg.T, cfg.E, cfg.d, cfg.h, cfg.k
        rows = E * c_stride(cfg)
        act = torch_dtype(cfg)
        self.stats = self._view(self.c.stats, (16,), torch.int32)
        r = self.c.route
        self.topk_idx = self._view(r.topk_idx, (T, k), torch.int32)
        self.counts = self._view(r.counts, (E,), torch.int32)
        self.slot_token = self._view(r.slot_token, (rows,), torch.int32)
        self.gate = self._view(r.gate, (rows,), torch.float32)
        self.tok_ptr = self._view(r.tok_ptr, (T + 1,), torch.int32)
        self.tok_row = self._view(r.tok_row, (rows,), torch.int32)
        self.delta = self._view(self.c.delta, (T, E), torch.float32)
        self.Z = self._view(self.c.Z, (T, d // cfg.D), torch.float32)
        self.xnorm = self._view(self.c.xnorm, (T,), torch.float32)
        self.rnorm = self._view(self.c.rnorm, (E,), torch.float32)
        for name, width in (("Xp", d), ("G", h), ("U", h), ("H", h), ("O", d), ("dO", d), ("dG", h),
                            ("dU", h), ("dXp", d)):
            setattr(self, name, self._view(getattr(self.c, name), (rows, width), act))
        self.dgate = self._view(self.c.dgate, (rows,), torch.float32)
        if host_staging:
            for name in ("X_dev", "dY_dev", "Y_dev", "dX_dev"):
                setattr(self, name, self._view(getattr(self.c, name), (T, d), act))
        if cfg.gate_mode == GATE_SOFTMAX:
            self.lse = self._view(self.c.lse, (T,), torch.float32)
            self.ddelta = self._view(self.c.ddelta, (T, E), torch.float32)

    def _view(self, ptr, shape, dtype):
        off = ptr - self.block.data_ptr()
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        return self.block[off:off + nbytes].view(dtype).view(*shape)

    @property
    def route(self) -> Route:
        return self.c.route

    def read_stats(self) -> Stats:
        return read_stats(self.c.stats)


def read_stats(stats_dev_ptr) -> Stats:
    s = Stats()
    code = lib().etr_read_stats(_p(stats_dev_ptr), C.byref(s), _stream())
    _check(code, "etr_read_stats")
    return s


def selftest_bounded_wait(stats, limit_cycles: int):
    """Launches the wait self-test: error_word of `stats` becomes non-zero after limit_cycles."""
    _check(lib().etr_selftest_bounded_wait(_p(stats), C.c_int64(int(limit_cycles)), _stream()),
           "etr_selftest_bounded_wait")


# ---- stage calls (same names as the C ABI) -------------------------------------------------
def affinity(cfg, X, R, delta, Z, xnorm, rnorm, stats):
    _check(lib().etr_affinity(C.byref(cfg), _p(X), _p(R), _p(delta), _p(Z), _p(xnorm), _p(rnorm),
                              _p(stats), _stream()), "etr_affinity")


def select(cfg, delta, stats, route: Route, ws):
    _check(lib().etr_select(C.byref(cfg), _p(delta), _p(stats), C.byref(route), _p(ws), _stream()),
           "etr_select")


SELECT_STATIC_MAX_ENTRIES = 4 * 1024 * 1024


def select_static(cfg, delta, stats, route: Route):
    """etr_select without a scratch argument: for callers that cannot allocate device memory.
    The keys live in a fixed 16 MiB array inside the library (T*E <= SELECT_STATIC_MAX_ENTRIES);
    calls that overlap on one GPU race on it."""
    _check(lib().etr_select_static(C.byref(cfg), _p(delta), _p(stats), C.byref(route), _stream()),
           "etr_select_static")


def dispatch(cfg, X, route: Route, Xp):
    _check(lib().etr_dispatch(C.byref(cfg), _p(X), C.byref(route), _p(Xp), _stream()), "etr_dispatch")


def expert_ffn(cfg, route: Route, Xp, W1g, W1u, W2, G, U, H, O, stats, ws):
    _check(lib().etr_expert_ffn(C.byref(cfg), C.byref(route), _p(Xp), _p(W1g), _p(W1u), _p(W2), _p(G),
                                _p(U), _p(H), _p(O), _p(stats), _p(ws), _stream()), "etr_expert_ffn")


def combine(cfg, route: Route, O, Y):
    _check(lib().etr_combine(C.byref(cfg), C.byref(route), _p(O), _p(Y), _stream()), "etr_combine")


def combine_bwd(cfg, route: Route, dY, O, dO, dgate):
    _check(lib().etr_combine_bwd(C.byref(cfg), C.byref(route), _p(dY), _p(O), _p(dO), _p(dgate),
                                 _stream()), "etr_combine_bwd")


def expert_ffn_bwd(cfg, route: Route, dO, Xp, G, U, H, W1g, W1u, W2, dG, dU, dXp, dW1g, dW1u, dW2,
                   stats, ws):
    _check(lib().etr_expert_ffn_bwd(C.byref(cfg), C.byref(route), _p(dO), _p(Xp), _p(G), _p(U), _p(H),
                                    _p(W1g), _p(W1u), _p(W2), _p(dG), _p(dU), _p(dXp), _p(dW1g),
                                    _p(dW1u), _p(dW2), _p(stats), _p(ws), _stream()),
           "etr_expert_ffn_bwd")


def dispatch_bwd(cfg, route: Route, dXp, dX):
    _check(lib().etr_dispatch_bwd(C.byref(cfg), C.byref(route), _p(dXp), _p(dX), _stream()),
           "etr_dispatch_bwd")


def select_bwd(cfg, route: Route, dgate):
    _check(lib().etr_select_bwd(C.byref(cfg), C.byref(route), _p(dgate)), "etr_select_bwd")


def affinity_bwd(cfg, X, R, delta, Z, xnorm, rnorm, route: Route, dgate, dX, dR, ws):
    _check(lib().etr_affinity_bwd(C.byref(cfg), _p(X), _p(R), _p(delta), _p(Z), _p(xnorm), _p(rnorm),
                                  C.byref(route), _p(dgate), _p(dX), _p(dR), _p(ws), _stream()),
           "etr_affinity_bwd")


def gate_softmax(cfg, delta, route: Route, lse):
    _check(lib().etr_gate_softmax(C.byref(cfg), _p(delta), C.byref(route), _p(lse), _stream()),
           "etr_gate_softmax")


def gate_softmax_bwd(cfg, delta, lse, route: Route, dgate, ddelta):
    _check(lib().etr_gate_softmax_bwd(C.byref(cfg), _p(delta), _p(lse), C.byref(route), _p(dgate),
                                      _p(ddelta), _stream()), "etr_gate_softmax_bwd")


def affinity_bwd_dense(cfg, X, R, delta, Z, xnorm, rnorm, route: Route, ddelta, dX, dR, ws):
    _check(lib().etr_affinity_bwd_dense(C.byref(cfg), _p(X), _p(R), _p(delta), _p(Z), _p(xnorm), _p(rnorm),
                                        C.byref(route), _p(ddelta), _p(dX), _p(dR), _p(ws), _stream()),
           "etr_affinity_bwd_dense")


def load_stats(cfg, route: Route, load, gate_mean):
    _check(lib().etr_load_stats(C.byref(cfg), C.byref(route), _p(load), _p(gate_mean), _stream()),
           "etr_load_stats")


def layer_forward(cfg, X, R, W1g, W1u, W2, buf: LayerBuffers, Y):
    _check(lib().etr_layer_forward(C.byref(cfg), _p(X), _p(R), _p(W1g), _p(W1u), _p(W2),
                                   C.byref(buf.c), _p(Y), _stream()), "etr_layer_forward")


def layer_backward(cfg, X, R, W1g, W1u, W2, dY, buf: LayerBuffers, dX, dR, dW1g, dW1u, dW2):
    _check(lib().etr_layer_backward(C.byref(cfg), _p(X), _p(R), _p(W1g), _p(W1u), _p(W2), _p(dY),
                                    C.byref(buf.c), _p(dX), _p(dR), _p(dW1g), _p(dW1u), _p(dW2),
                                    _stream()), "etr_layer_backward")


class HostSlotC(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("X_dev", "dY_dev", "Y_dev", "dX_dev")]


HOST_SLOTS = 4


class HostSlot:
    """Device staging of one host step in flight (four [T, d] tensors of the activation dtype)."""

    def __init__(self, cfg: Config, index: int, device="cuda"):
        self.index = index
        self.tensors = [torch.empty(cfg.T, cfg.d, dtype=torch_dtype(cfg), device=device) for _ in range(4)]
        self.c = HostSlotC(*[C.c_void_p(t.data_ptr()) for t in self.tensors])


def layer_step_host_begin(cfg, X_host, dY_host, R, W1g, W1u, W2, buf: "LayerBuffers", slot: HostSlot,
                          Y_host, dX_host, dR, dW1g, dW1u, dW2):
    """Enqueues one step from host tensors on `slot` and returns without waiting."""
    _check(lib().etr_layer_step_host_begin(C.byref(cfg), _p(X_host), _p(dY_host), _p(R), _p(W1g), _p(W1u),
                                           _p(W2), C.byref(buf.c), C.byref(slot.c), C.c_int32(slot.index),
                                           _p(Y_host), _p(dX_host), _p(dR), _p(dW1g), _p(dW1u), _p(dW2),
                                           _stream()), "etr_layer_step_host_begin")


def layer_step_host_wait(slot: HostSlot):
    _check(lib().etr_layer_step_host_wait(C.c_int32(slot.index)), "etr_layer_step_host_wait")


def layer_step_host(cfg, X_host, dY_host, R, W1g, W1u, W2, buf: LayerBuffers, Y_host, dX_host, dR,
                    dW1g, dW1u, dW2):
    """X_host, dY_host, Y_host, dX_host are CPU tensors (pinned for full copy speed)."""
    _check(lib().etr_layer_step_host(C.byref(cfg), _p(X_host), _p(dY_host), _p(R), _p(W1g), _p(W1u),
                                     _p(W2), C.byref(buf.c), _p(Y_host), _p(dX_host), _p(dR),
                                     _p(dW1g), _p(dW1u), _p(dW2), _stream()), "etr_layer_step_host")
