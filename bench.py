"""Benchmark of the ETR MoE layer: forward + backward tokens/s on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large] [--impl reference]

A step is one pass of the whole hot path (affinity, selection, dispatch, expert FFN,
combine and every backward stage) over one batch of seeded synthetic tokens.  With N > 1
(launched by torch.distributed.run) every rank runs an independent replica of the layer on
its own tokens: the path has no exchange step, so there is no data-path collective and the
scaling is weak.  Rank 0 prints one JSON line.

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from gen import workloads as gw  # noqa: E402

METRIC = "etr_moe_layer_fwd_bwd_tokens_per_sec"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised
# under profiles/ (absent: not captured for the current version of that kernel).
NCU_TRAFFIC_BYTES = {}
# tc_grouped_gemm_pair_kernel and its wide form: measured on the mid workload, all 7 launches of one step
# (profiles/tc_grouped_gemm_pair_kernels_mid_ncu_full.md): 3674.3 MB of DRAM traffic against 3799.7 MB
# of algorithmic bytes (part of the output is still in L2 when a kernel ends).  The large workload is
# too big for a multi-pass capture, so its traffic is this ratio times its own algorithmic bytes.
TC_GEMM_DRAM_OVER_ALGORITHMIC = 3674.3 / 3799.7


def tc_gemm_algorithmic_bytes(w, rows_padded):
    """Bytes the seven grouped GEMMs of one step must move (bf16): activations once per use, every
    expert weight once per GEMM that reads it, every output once."""
    ad, ah, wt = rows_padded * w.d * 2, rows_padded * w.h * 2, w.E * w.d * w.h * 2
    reads = (ad + 2 * wt) + (ah + wt) + (ad + wt + 2 * ah) + (2 * ah + 2 * wt) + (ad + ah) + 2 * (ah + ad)
    writes = 3 * ah + ad + 2 * ah + ad + wt + 2 * wt
    return reads + writes


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


def mode_name(w):
    if w.mode in ("tcr", "ecr"):
        return w.mode
    return "tcr" if w.step < w.switch_step else "ecr"


# ---- algorithmic work per kernel and step (what the method itself must move / compute) ----
def algorithmic_work(w, rows, kernel, unrouted=0):
    """(amount, "bytes"|"flops") for all launches of `kernel` in one step."""
    b = 2 if w.dtype == "bf16" else 4
    T, d, E, h, m = w.T, w.d, w.E, w.h, w.m
    T_routed = T - unrouted
    table = {
        "affinity_fwd_kernel": (T * d * b + T * E * 4 + T * m * 4 + T * 4, "bytes"),
        "affinity_fwd_warp_kernel": (T * d * b + T * E * 4 + T * m * 4 + T * 4, "bytes"),
        "grap_pool_kernel": (T * d * b + T * m * 4 + T * 4, "bytes"),
        "affinity_score_kernel": (2 * T * m * E, "fp32_flops"),        # the product z R^T: fp32 FMA issue, not HBM
        "affinity_score_tc_kernel": (T * m * 4 + T * E * 4 + T * 4, "bytes"),   # the same product on the tensor cores
        "select_token_side_kernel": (2 * T * E * 4, "bytes"),
        "select_expert_side_kernel": (T * E * 4 + rows * 8, "bytes"),
        "csr_count_kernel": (T * E * 4, "bytes"),
        "csr_scan_kernel": (T * 8, "bytes"),
        "csr_fill_kernel": (T * E * 4 + rows * 4, "bytes"),
        "dispatch_kernel": (2 * rows * d * b, "bytes"),
        "combine_kernel": (rows * d * b + T * d * b, "bytes"),
        "zero_unrouted_kernel": (unrouted * d * b + T * 4, "bytes"),
        "select_threshold_limit_kernel": (4 * T * E * 4, "bytes"),
        "combine_bwd_kernel": (3 * rows * d * b, "bytes"),
        "affinity_bwd_dx_kernel": (3 * T_routed * d * b, "bytes"),
        "affinity_bwd_dx_fused_kernel": (T_routed * d * b + rows * d * b + T * d * b, "bytes"),
        "affinity_bwd_dr_partial_kernel": (rows * m * 4, "bytes"),
        "affinity_bwd_dr_final_kernel": (E * m * 8, "bytes"),
        "affinity_bwd_dr_dense_partial_kernel": (T * m * 4 + T * E * 8, "bytes"),
        "gate_softmax_kernel": (T * E * 4 + rows * 12 + T * 4, "bytes"),
        "gate_softmax_bwd_kernel": (2 * T * E * 4 + rows * 12, "bytes"),
        "load_stats_kernel": (rows * 4, "bytes"),
        "gemm_simt_kernel": (18 * rows * d * h, "flops"),
        # tcgen05 grouped GEMMs: selected rows only (not the rows padding a 128-row tile)
        "tc_gemm_swiglu": (4 * rows * d * h, "flops"),
        "tc_gemm_down": (2 * rows * d * h, "flops"),
        "tc_gemm_dswiglu": (2 * rows * d * h, "flops"),
        "tc_gemm_dxp": (4 * rows * d * h, "flops"),
        "tc_gemm_dw2": (2 * rows * d * h, "flops"),
        "tc_gemm_dw1": (4 * rows * d * h, "flops"),
    }
    return table.get(kernel, (0, "bytes"))


def aggregate_over_ranks(values, world, device=None):
    """Element-wise max of per-rank timings over all ranks (the slowest rank sets the pace)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_tokens_per_sec(world, tokens_per_rank, ms_per_step):
    """Replicas process world * tokens_per_rank tokens per step (weak scaling)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample_run(w, inputs_host, weights_host, Ts, steps, warmup, threads=None, gpu_routing=None):
    """Times the CPU oracle (as it stands) on the first Ts tokens of the workload, all experts.

    The sample's capacity is scaled so that it does the same work per token as the full step when the
    full step's routing is known (gpu_routing = (C, rows, T)): C_sample = max(1, round(C * Ts / T)),
    fixed, not adaptive.  Otherwise the workload's own rule on Ts tokens."""
    from oracle import binding as ob
    cores = ob.set_threads(threads or os.cpu_count() or 1)
    o = ob.Oracle("f32")
    X, dY, R = inputs_host["X"][:Ts], inputs_host["dY"][:Ts], inputs_host["R"]
    W1g, W1u, W2 = weights_host
    mode = ob.MODE_TCR if mode_name(w) == "tcr" else ob.MODE_ECR
    if gpu_routing is not None:
        C_gpu, rows_gpu, T_gpu = gpu_routing
        capacity, adaptive = max(1, int(round(C_gpu * Ts / T_gpu))), False
    else:
        capacity, adaptive = replace(w, T=Ts).capacity, w.adaptive
    times, rows = [], 0
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        fw = o.forward(X, R, W1g, W1u, W2, D=w.D, k=w.k, capacity=capacity, mode=mode, adaptive=adaptive)
        o.backward(fw, X, R, W1g, W1u, W2, dY)
        rows = int(fw.route.tok_ptr[-1])
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    note = ""
    if gpu_routing is not None:
        note = f" (the full step: {gpu_routing[1] / gpu_routing[2]:.2f} rows per token at C={gpu_routing[0]})"
    return {"value": Ts / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
            "rows_per_token": rows / Ts,
            "sample": f"first {Ts} tokens of the workload, all {w.E} experts, capacity {capacity}: "
                      f"{rows} rows = {rows / Ts:.2f} rows per token{note}, full forward+backward, "
                      f"{len(times)} step(s) of {sec:.2f} s on {cores} thread(s)"}, sec


def device_weights(w, device, seed):
    """Expert weights ~ N(0, 1/d) drawn on the device (seeded); bf16 or fp32 per workload."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    std = 1.0 / np.sqrt(w.d)
    out = []
    for shape in ((w.E, w.h, w.d), (w.E, w.h, w.d), (w.E, w.d, w.h)):
        t = torch.empty(shape, dtype=dt, device=device)
        for e in range(w.E):                       # per expert: bounded fp32 temporaries
            t[e] = (torch.randn(shape[1:], generator=g, device=device) * std).to(dt)
        out.append(t)
    return out


GEMM_IMPLS = {"auto": "GEMM_AUTO", "simt": "GEMM_SIMT", "tcgen05": "GEMM_TCGEN05",
              "tcgen05_2cta": "GEMM_TCGEN05_2CTA", "tcgen05_2cta_wide": "GEMM_TCGEN05_2CTA_WIDE"}


class Layer:
    """One layer instance on the device: inputs, parameters, buffers, outputs, and `step()`."""

    def __init__(self, etr, w, dev, args, inp=None, weights=None, host_staging=False, delta_max_override=-1.0,
                 adaptive=None):
        self.etr, self.w = etr, w
        inp = inp if inp is not None else gw.make_inputs(w, weights=False)
        self.inp = inp
        act = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        self.Xh = torch.from_numpy(inp["X"]).to(act)
        self.dYh = torch.from_numpy(inp["dY"]).to(act)
        self.X, self.dY = self.Xh.to(dev), self.dYh.to(dev)
        self.R = torch.from_numpy(inp["R"]).to(dev)
        self.W1g, self.W1u, self.W2 = weights if weights is not None else device_weights(w, dev, w.seed)
        self.cfg = etr.make_config(
            T=w.T, d=w.d, D=w.D, E=w.E, k=w.k, h=w.h, capacity=w.capacity,
            dtype=etr.BF16 if w.dtype == "bf16" else etr.F32,
            mode=etr.MODE_TCR if mode_name(w) == "tcr" else etr.MODE_ECR, step=w.step, switch_step=w.switch_step,
            adaptive=w.adaptive if adaptive is None else adaptive, delta_max_override=delta_max_override,
            gemm_impl=getattr(etr, GEMM_IMPLS[args.gemm]),
            fuse_dispatch={"auto": etr.FUSE_AUTO, "off": etr.FUSE_OFF, "on": etr.FUSE_ON}[args.fuse],
            gate_mode=etr.GATE_SOFTMAX if args.gate == "softmax" else etr.GATE_AFFINITY)
        self.buf = etr.LayerBuffers(self.cfg, host_staging=host_staging, device=dev)
        self.Y, self.dX = torch.empty_like(self.X), torch.empty_like(self.X)
        self.dR = torch.empty_like(self.R)
        self.dW1g, self.dW1u, self.dW2 = (torch.empty_like(t) for t in (self.W1g, self.W1u, self.W2))

    def step(self):
        e = self.etr
        e.layer_forward(self.cfg, self.X, self.R, self.W1g, self.W1u, self.W2, self.buf, self.Y)
        e.layer_backward(self.cfg, self.X, self.R, self.W1g, self.W1u, self.W2, self.dY, self.buf, self.dX,
                         self.dR, self.dW1g, self.dW1u, self.dW2)


def timed_steps(layer, n, barrier):
    """n steps back to back, one CUDA-event pair around all of them (on the launch stream)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(n):
        layer.step()
    e1.record()
    barrier()
    return e0.elapsed_time(e1)


def graph_ms_per_step(layer, n, barrier):
    """One step captured in a CUDA graph (the calls enqueue stream work only) and replayed n times."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        layer.step()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        layer.step()
    g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(n):
        g.replay()
    e1.record()
    barrier()
    return e0.elapsed_time(e1) / n


def per_kernel_pass(etr, layer, n, barrier):
    """n more steps with an event pair around every launch; [(kernel, ms)]."""
    etr.timing_enable(True)
    for _ in range(n):
        layer.step()
    barrier()
    recs = etr.timing_collect()
    etr.timing_enable(False)
    return recs


def kernel_table(w, recs, rows, unrouted, steps, peaks, tensor_peak, sm_max_mhz, dev):
    per = {}
    for name, ms in recs:
        if ms >= 0:
            a = per.setdefault(name, [0, 0.0])
            a[0] += 1
            a[1] += ms
    total = sum(v[1] for v in per.values()) or 1.0
    kernels = []
    for name, (n, ms) in sorted(per.items(), key=lambda kv: -kv[1][1]):
        amount, kind = algorithmic_work(w, rows, name, unrouted)
        per_launch = amount * steps / n if n else 0.0
        avg_ms = ms / n
        if kind == "flops":
            ach, peak, unit, bound = per_launch / (avg_ms * 1e-3) / 1e12, tensor_peak, "TFLOP/s", "tensor"
        elif kind == "fp32_flops":
            # plain fp32 multiply-adds: SMs x 128 lanes x 2 flop at the maximum SM clock (nominal, not measured)
            sms = torch.cuda.get_device_properties(dev).multi_processor_count
            peak = sms * 128 * 2 * (sm_max_mhz or 1965.0) * 1e6 / 1e12
            ach, unit, bound = per_launch / (avg_ms * 1e-3) / 1e12, "TFLOP/s", "alu"
        else:
            ach, peak, unit, bound = per_launch / (avg_ms * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
        kernels.append({"kernel": name, "launches_per_step": n / steps, "ms_per_step": ms / steps,
                        "share": ms / total, "bound": bound, "achieved": ach, "peak": peak, "unit": unit,
                        "frac": ach / peak})
    return kernels


def gemm_summary(w, kernels, rows):
    """(TFLOP/s over all tensor-core launches, their ms per step, launches per step, flops per step)."""
    tc = [k for k in kernels if k["kernel"].startswith("tc_gemm_")]
    if not tc:
        return None
    flops = sum(algorithmic_work(w, rows, k["kernel"])[0] for k in tc)
    ms = sum(k["ms_per_step"] for k in tc)
    n = sum(k["launches_per_step"] for k in tc)
    return {"tflops": flops / (ms * 1e-3) / 1e12, "ms_per_step": ms, "launches_per_step": n, "flops_per_step": flops,
            "share_of_step": ms / (sum(k["ms_per_step"] for k in kernels) or 1.0)}


def measure_other(etr, name, w, dev, args, barrier, peaks, inp=None, weights=None, delta_max_override=-1.0,
                  adaptive=None, steps=10):
    """A short device-timed measurement of another workload: ms per step, tokens/s, routing, GEMM rate."""
    layer = Layer(etr, w, dev, args, inp=inp, weights=weights, delta_max_override=delta_max_override,
                  adaptive=adaptive)
    for _ in range(3):
        layer.step()
    barrier()
    st = layer.buf.read_stats()
    ms = timed_steps(layer, steps, barrier) / steps
    kernels = kernel_table(w, per_kernel_pass(etr, layer, steps, barrier), st.rows_total, st.unrouted, steps, peaks,
                           peaks["bf16_tflops"], None, dev)
    ms_graph = graph_ms_per_step(layer, steps, barrier)
    assert layer.buf.read_stats().error_word == 0
    g = gemm_summary(w, kernels, st.rows_total)
    out = {"workload": name, "T": w.T, "mode": mode_name(w), "C": st.C, "capacity": w.capacity,
           "rows": st.rows_total, "unrouted": st.unrouted, "delta_max": st.delta_max, "steps": steps,
           "ms_per_step": ms, "tokens_per_s": w.T / (ms * 1e-3), "ms_per_step_cuda_graph": ms_graph}
    if g:
        out.update(gemm_tflops=g["tflops"], gemm_frac_of_burst_peak=g["tflops"] / peaks["bf16_tflops"],
                   gemm_share_of_step=g["share_of_step"])
    return out, layer


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=list(gw.WORKLOADS))
    ap.add_argument("--gemm", default="auto", choices=list(GEMM_IMPLS))
    ap.add_argument("--fuse", default="auto", choices=["auto", "off", "on"],
                    help="token rearrangement fused into the GEMM operand fetch (TMA row gathers)")
    ap.add_argument("--gate", default="affinity", choices=["affinity", "softmax"],
                    help="gate of a selected pair: raw affinity (default) or softmax over the experts")
    ap.add_argument("--cpu-tokens", type=int, default=256, help="tokens in the all-cores CPU-oracle sample")
    ap.add_argument("--cpu-tokens-single", type=int, default=64, help="tokens in the single-thread CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustain-seconds", type=float, default=3.0,
                    help="length of the sustained pass (0: skip it)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the short measurements of the other workloads (they run at N=1 only)")
    ap.add_argument("--set", default="", help="override workload fields, e.g. T=32768,h=512 (profiling cases)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    w0 = gw.WORKLOADS[args.workload]
    if args.set:
        kv = dict(item.split("=") for item in args.set.split(","))
        w0 = replace(w0, name=w0.name + "+" + args.set,
                     **{k: type(getattr(w0, k))(v) for k, v in kv.items()})
    config = {"workload": f"{w0.name} (config {w0.config_id}): T={w0.T} d={w0.d} D={w0.D} E={w0.E} "
                          f"k={w0.k} h={w0.h} cf={w0.cf} {mode_name(w0)} adaptive={int(w0.adaptive)} "
                          f"x={w0.x_kind}",
              "T": w0.T, "d": w0.d, "D": w0.D, "E": w0.E, "k": w0.k, "h": w0.h,
              "capacity": w0.capacity, "mode": mode_name(w0), "adaptive": bool(w0.adaptive),
              "l2": "inputs larger than L2 (no flush)", "parallelism": f"replicas x{world}"}

    if args.impl == "reference":
        if rank != 0:
            return
        w = w0
        Ts = min(args.cpu_tokens, w.T)
        routing = None
        if w.adaptive and Ts < w.T:
            # The capacity the whole batch gives (its maximum affinity sets the adaptive bound), from the
            # oracle's own affinity pass over all T tokens, so that the sample does the work per token of
            # the full step; the timed steps then run on the first Ts tokens.
            from oracle import binding as ob
            ob.set_threads(os.cpu_count() or 1)
            full = gw.make_inputs(w, weights=False)
            _, _, _, dmax = ob.Oracle("f32").affinity(full["X"], full["R"], w.D)
            C = ob.capacity_bound(w.d, w.E, w.capacity, 1, True, float(dmax))
            mode = ob.MODE_TCR if mode_name(w) == "tcr" else ob.MODE_ECR
            rows = min(C, w.T) * w.E if mode == ob.MODE_ECR else None
            inp = {"X": full["X"][:Ts].copy(), "dY": full["dY"][:Ts].copy(), "R": full["R"]}
            del full
            if rows is not None:
                routing = (C, rows, w.T)
        else:
            inp = gw.make_inputs(replace(w, T=Ts), weights=False)
            inp["R"] = gw.expert_embeddings(w)
        W = gw.expert_weights(w)
        base, sec = oracle_sample_run(w, inp, W, Ts, max(1, args.steps), args.warmup, gpu_routing=routing)
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}))
        return

    from paper_2406_00023_b200 import etr
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    w = replace(w0, config_id=w0.config_id + 1000 * rank)       # each replica: its own tokens

    layer = Layer(etr, w, dev, args, host_staging=True)
    cfg, buf, inp = layer.cfg, layer.buf, layer.inp
    Xh, dYh = layer.Xh.pin_memory(), layer.dYh.pin_memory()
    Yh, dXh = torch.empty_like(Xh).pin_memory(), torch.empty_like(Xh).pin_memory()
    R, W1g, W1u, W2 = layer.R, layer.W1g, layer.W1u, layer.W2
    dR, dW1g, dW1u, dW2 = layer.dR, layer.dW1g, layer.dW1u, layer.dW2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        layer.step()
    barrier()
    st = buf.read_stats()
    assert st.error_word == 0, "a device-side wait expired during warm-up"
    rows = st.rows_total
    rows_padded = int(((buf.counts.cpu().numpy() + 127) // 128 * 128).sum())
    peaks = load_peaks()

    # Pass 1, the reported value: K steps back to back, one event pair around all of them.
    sampler = ClockSampler(local)
    sampler.start()
    n0 = etr.launch_count()
    ms_total = timed_steps(layer, args.steps, barrier)
    launches = etr.launch_count() - n0
    # Pass 2, the per-kernel table and the roofline: K more steps with an event pair around every
    # launch (the pairs cost a few percent of the step, which is why pass 1 runs without them).
    recs = per_kernel_pass(etr, layer, args.steps, barrier)
    clocks = sampler.stop()
    assert buf.read_stats().error_word == 0

    # Pass 3, sustained: the same step repeated for several seconds, until the power cap has pulled the
    # SM clock down to where a training loop runs, then a per-kernel pass from that state.
    sustained, recs_hot = None, None
    if args.sustain_seconds > 0:
        n_long = max(args.steps, int(np.ceil(args.sustain_seconds * 1e3 / (ms_total / args.steps))))
        hot = ClockSampler(local)
        hot.start()
        ms_long = timed_steps(layer, n_long, barrier)
        recs_hot = per_kernel_pass(etr, layer, args.steps, barrier)
        hot_clocks = hot.stop()
        assert buf.read_stats().error_word == 0
        sustained = {"steps": n_long, "seconds": ms_long * 1e-3, "ms_per_step": ms_long / n_long,
                     "sm_mhz_median": hot_clocks.get("sm_mhz"), "reasons": hot_clocks.get("reasons"),
                     "clock_samples": hot_clocks.get("samples")}

    # End to end through the host-buffer entry points (H2D and D2H of every step inside the timed
    # region).  First one step at a time (etr_layer_step_host: returns when Y and dX are on the
    # host), then the loop form a training loop uses (etr_layer_step_host_begin/_wait on two
    # slots: the next step's uploads run under this step's kernels).
    e2e_steps = max(1, min(args.steps, 5))
    etr.layer_step_host(cfg, Xh, dYh, R, W1g, W1u, W2, buf, Yh, dXh, dR, dW1g, dW1u, dW2)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        etr.layer_step_host(cfg, Xh, dYh, R, W1g, W1u, W2, buf, Yh, dXh, dR, dW1g, dW1u, dW2)
    torch.cuda.synchronize()
    e2e_single_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps

    slots = [etr.HostSlot(cfg, i, device=dev) for i in range(2)]
    for i in range(2):
        etr.layer_step_host_begin(cfg, Xh, dYh, R, W1g, W1u, W2, buf, slots[i], Yh, dXh, dR, dW1g, dW1u, dW2)
    for sl in slots:
        etr.layer_step_host_wait(sl)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        sl = slots[i % 2]
        etr.layer_step_host_wait(sl)          # the step that used this slot two steps ago has delivered
        etr.layer_step_host_begin(cfg, Xh, dYh, R, W1g, W1u, W2, buf, sl, Yh, dXh, dR, dW1g, dW1u, dW2)
    for sl in slots:
        etr.layer_step_host_wait(sl)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / args.steps
    del slots

    agg = [ms_total, e2e_ms, e2e_single_ms] + ([sustained["ms_per_step"]] if sustained else [])
    agg = aggregate_over_ranks(agg, world, dev)
    ms_total, e2e_ms, e2e_single_ms = agg[:3]
    if sustained:
        sustained["ms_per_step"] = agg[3]
        sustained["tokens_per_s"] = whole_job_tokens_per_sec(world, w.T, agg[3])
    ms_step = ms_total / args.steps

    # Per-kernel table and the roofline of the dominant kernel.  The short passes run near the maximum
    # clock, so their tensor-core rate is set against the measured burst peak; the sustained pass runs
    # power-capped, like the loop behind the measured sustained peak, and is set against that one.
    kernels = kernel_table(w, recs, rows, st.unrouted, args.steps, peaks, peaks["bf16_tflops"],
                           clocks.get("sm_max_mhz"), dev)
    kernels_hot = (kernel_table(w, recs_hot, rows, st.unrouted, args.steps, peaks, peaks["bf16_tflops_sustained"],
                                clocks.get("sm_max_mhz"), dev) if recs_hot else None)
    g = gemm_summary(w, kernels, rows)
    roofline = None
    if g and g["share_of_step"] >= 0.5:
        # The six tcgen05 contractions run on one persistent grouped-GEMM design in two tile forms
        # (--gemm can force one); the roofline entry covers all their launches.
        pair = args.gemm == "auto"          # the ncu traffic ratio was taken with the library's own choice
        kname = {"auto": "tc_grouped_gemm_pair_kernel + tc_grouped_gemm_pair_wide_kernel (chosen per contraction)",
                 "tcgen05_2cta": "tc_grouped_gemm_pair_kernel", "tcgen05_2cta_wide": "tc_grouped_gemm_pair_wide_kernel",
                 "tcgen05": "tc_grouped_gemm_kernel"}.get(args.gemm, "tc_grouped_gemm")
        roofline = {"kernel": kname, "launches_per_step": g["launches_per_step"], "bound": "tensor",
                    "achieved": g["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": g["tflops"] / peaks["bf16_tflops"],
                    "flops_per_launch": g["flops_per_step"] / g["launches_per_step"],
                    "avg_launch_ms": g["ms_per_step"] / g["launches_per_step"],
                    "traffic": (TC_GEMM_DRAM_OVER_ALGORITHMIC * tc_gemm_algorithmic_bytes(w, rows_padded)
                                / g["launches_per_step"] if pair else None),
                    "traffic_note": "ncu dram bytes of the mid workload scaled by algorithmic bytes",
                    "peak_source": peaks["source"] + " (burst: the timed passes last a fraction of a second)"}
        if kernels_hot:
            gh = gemm_summary(w, kernels_hot, rows)
            roofline["sustained"] = {"achieved": gh["tflops"], "peak": peaks["bf16_tflops_sustained"],
                                     "frac": gh["tflops"] / peaks["bf16_tflops_sustained"],
                                     "avg_launch_ms": gh["ms_per_step"] / gh["launches_per_step"],
                                     "peak_source": peaks["source"] + " (sustained: per-kernel pass after "
                                                    f"{sustained['seconds']:.1f} s of steps)"}
    elif kernels:
        top = kernels[0]
        roofline = {"kernel": top["kernel"], "bound": top["bound"], "achieved": top["achieved"],
                    "peak": top["peak"], "unit": top["unit"], "frac": top["frac"],
                    "traffic": NCU_TRAFFIC_BYTES.get(top["kernel"]),
                    "peak_source": peaks["source"] + (" (burst)" if top["bound"] == "tensor" else "")}

    out = {"metric": METRIC, "value": whole_job_tokens_per_sec(world, w.T, ms_step), "unit": UNIT, "n_gpus": world,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic", "config": config,
           "clocks": clocks, "gpu_launches": int(launches),
           "e2e": {"value": whole_job_tokens_per_sec(world, w.T, e2e_ms), "unit": UNIT,
                   "h2d_bytes_per_step": int(2 * Xh.numel() * Xh.element_size()),
                   "d2h_bytes_per_step": int(2 * Xh.numel() * Xh.element_size()),
                   "ms_per_step": e2e_ms, "how": "K steps through etr_layer_step_host_begin/_wait on two slots",
                   "ms_per_step_one_at_a_time": e2e_single_ms},
           "roofline": roofline, "sustained": sustained, "kernels": kernels, "kernels_sustained": kernels_hot,
           "kernel_timing": "a second pass of the same K steps with a CUDA-event pair around every launch",
           "routing": {"C": st.C, "rows": rows, "dropped": st.dropped, "unrouted": st.unrouted,
                       "delta_max": st.delta_max}}

    if rank == 0 and world == 1 and not args.no_other_workloads:
        out["other_workloads"] = other_workloads(etr, layer, dev, args, barrier, peaks)

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        Wh = [t.float().cpu().numpy() for t in (W1g, W1u, W2)]
        host = {"X": inp["X"], "dY": inp["dY"], "R": inp["R"]}
        routing = (st.C, rows, w.T)
        base, _ = oracle_sample_run(w, host, Wh, min(args.cpu_tokens, w.T), 1, 0, gpu_routing=routing)
        single, _ = oracle_sample_run(w, host, Wh, min(args.cpu_tokens_single, w.T), 1, 0, threads=1,
                                      gpu_routing=routing)
        base["single_thread"] = single
        out["cpu_baseline"] = base
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def other_workloads(etr, main_layer, dev, args, barrier, peaks):
    """Short device-timed runs of the workloads the headline does not time: tiny, small, mid, the eight
    points of the adaptive-switch sweep (each with the measured delta_max and with the supplied
    delta_max schedule that walks C through the interior of its clamp), and the main workload at full
    capacity (adaptive bound off)."""
    res = []
    w_main = main_layer.w
    if w_main.adaptive:      # same tensors, the adaptive bound switched off: every expert filled to `capacity`
        r, lay = measure_other(etr, f"{w_main.name}, adaptive bound off (C = capacity)", w_main, dev, args, barrier,
                               peaks, inp=main_layer.inp, weights=(main_layer.W1g, main_layer.W1u, main_layer.W2),
                               adaptive=False)
        res.append(r)
        del lay
    torch.cuda.empty_cache()
    for name in ("tiny", "small", "mid"):
        if name == w_main.name:
            continue
        r, lay = measure_other(etr, name, gw.WORKLOADS[name], dev, args, barrier, peaks)
        res.append(r)
        del lay
    if w_main.name != "sweep":
        sw = gw.WORKLOADS["sweep"]
        weights = device_weights(sw, dev, sw.seed)
        R = gw.expert_embeddings(sw)
        dY = gw.output_grad(sw)
        for i, step in enumerate(gw.SWEEP_STEPS):
            wp = gw.sweep_point(i)
            inp = {"R": R, "X": gw.tokens(wp, R), "dY": dY}
            for label, ov in (("measured delta_max", -1.0), (f"delta_max {gw.SWEEP_DELTA_MAX[i]}", gw.SWEEP_DELTA_MAX[i])):
                r, lay = measure_other(etr, f"sweep step {step} ({label})", wp, dev, args, barrier, peaks, inp=inp,
                                       weights=weights, delta_max_override=ov, steps=5)
                res.append(r)
                del lay
    torch.cuda.empty_cache()
    return res


if __name__ == "__main__":
    main()
