#!/usr/bin/env python
"""Benchmark of the dai8 hot path on one B200 (or N independent replicas, one per GPU).

Workload: the ResNet-50 conv2_x bottleneck block (1x1 256->64, 3x3 64->64 pad 1, 1x1 64->256) at
N=64, 56x56, bf16 NHWC inputs, synthetic tensors (X = ReLU(N(0,1)), He weights, per-channel
bell-shaped / long-tailed dY).  One step = the whole path for the three layers: forward
quantization of X and W, int8 forward conv, gradient vectorized quantization of dY (statistics,
density count, clip update, vq + gq codes), int8 dW and dX convs with de-quantizing epilogues.

Prints ONE JSON line.  `value` = int8 backward-convolution throughput, 2*MACs(dX+dW) of the step
divided by the time of the WHOLE step (quantization and the forward conv included), in TOPS, summed
over ranks.  `detail` holds the per-call breakdown measured with CUDA events in a second pass of the same
steps, `roofline` the dominant call, `e2e` the same metric with pinned-host inputs and outputs
copied inside the timed region, `cpu_baseline` the CPU oracle on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "int8 conv-backward TOPS (dX+dW)"
UNIT = "TOPS"
WORKLOAD = "resnet50_conv2x_bottleneck_N64_56x56_bf16_nhwc"
BATCH = 64
SEED = 2024
INT8_OVER_BF16 = 2.0   # nominal dense ratio 4.5 / 2.25 PFLOP/s
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant call's kernel, from the ncu
# capture summarised in profiles/gvq_fused_nhwc_bf16_conv2x.md (bytes; None once the kernel changes)
NCU_TRAFFIC = {"quantize_grad @ conv2_x.1x1b": 189.12e6 + 58.67e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_step(inputs):
    """The whole path for a list of (layer, x, w, g) with the CPU oracle, as it stands."""
    from oracle import cpu as O
    for L, x, w, g in inputs:
        sx, sw = float(np.abs(x).max()), float(np.abs(w).max())
        qx, qw = O.quantize(x, sx), O.quantize(w, sw)
        O.dequant_acc(O.conv_fwd_acc(qx, qw, L.stride, L.pad)[0], sx, sw)
        absmax, _, sigma, gl = O.channel_stats(g)
        cnt = O.density_count(g, sigma)
        s, _ = O.classify_clip(cnt, absmax, g.size // g.shape[1])
        vq = O.quantize(g, s, True, SEED, 0)
        gq = O.quantize(g, gl, True, SEED, 1)
        O.dequant_acc(O.conv_bwd_filter_acc(qx, vq, (L.R, L.S), L.stride, L.pad)[0], sx, s)
        O.dequant_acc(O.conv_bwd_data_acc(gq, qw, (L.H, L.W), L.stride, L.pad)[0], gl, sw)


def oracle_inputs(batch):
    from paper_2102_04782_b200 import synth
    out = []
    for i, L in enumerate(synth.resnet50_conv2x_block()):
        x, w, g, _, _ = synth.layer_inputs(L, batch, SEED + i, bf16=True)
        out.append((L, x, w, g))
    return out


def bwd_ops(layers, batch):
    return sum(2 * 2 * L.macs(batch) for L in layers)   # dX + dW, 2 ops per MAC


def time_oracle(batch, steps, warmup):
    from oracle import cpu as O
    from paper_2102_04782_b200 import synth
    inputs = oracle_inputs(batch)
    for _ in range(warmup):
        oracle_step(inputs)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(inputs)
    dt = (time.perf_counter() - t0) / steps
    ops = bwd_ops(synth.resnet50_conv2x_block(), batch)
    return ops / dt / 1e12, dt, O.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    batch = 4
    value, dt, cores = time_oracle(batch, args.steps, args.warmup)
    sample = f"same three layers at batch {batch} of {BATCH} per step (bounded sample), CPU oracle as it stands"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# Multi-GPU: replicas only.  Every rank runs the whole workload on its own GPU; the only exchange
# is the timing itself (max over ranks) and rank 0 prints the aggregate.  These two helpers hold
# that logic so that it can be exercised with the gloo backend on CPU.
# ------------------------------------------------------------------------------------------------
def max_over_ranks(ms, dist=None, device="cpu"):
    """Slowest rank's time in milliseconds (the job is as slow as its slowest replica)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(ops_per_step_per_rank, ms_per_step, world):
    """Whole-job TOPS of `world` replicas that each do ops_per_step_per_rank in ms_per_step."""
    return world * ops_per_step_per_rank / (ms_per_step * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------
class LayerBuffers:
    def __init__(self, L, N, seed, torch, api, synth, dev):
        self.L, self.N = L, N
        x, w, g, _, _ = synth.layer_inputs(L, N, seed, bf16=True)
        bf = torch.bfloat16
        self.h_x = torch.from_numpy(x).permute(0, 2, 3, 1).contiguous().to(bf).pin_memory()
        self.h_w = torch.from_numpy(w).to(bf).pin_memory()
        self.h_g = torch.from_numpy(g).permute(0, 2, 3, 1).contiguous().to(bf).pin_memory()
        self.x, self.w, self.g = self.h_x.to(dev), self.h_w.to(dev), self.h_g.to(dev)
        self.geom = api.ConvGeom(N, L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.stride, L.pad, L.pad)
        Cip, Cop = api.padded_channels(L.Cin), api.padded_channels(L.Cout)
        i8 = dict(dtype=torch.int8, device=dev)
        f32 = dict(dtype=torch.float32, device=dev)
        self.qX = torch.empty((N, L.H, L.W, Cip), **i8)
        self.qW = torch.empty((L.Cout, L.R, L.S, Cip), **i8)
        self.vq = torch.empty((N, L.P, L.Q, Cop), **i8)
        self.gq = torch.empty((N, L.P, L.Q, Cop), **i8)
        self.sX, self.sW, self.gmax = torch.zeros(1, **f32), torch.zeros(1, **f32), torch.zeros(1, **f32)
        self.s_state = torch.zeros(L.Cout, **f32)
        self.Y = torch.empty((N, L.P, L.Q, L.Cout), dtype=bf, device=dev)
        self.dX = torch.empty((N, L.H, L.W, L.Cin), dtype=bf, device=dev)
        self.dW = torch.empty((L.Cout, L.Cin, L.R, L.S), **f32)
        u8 = dict(dtype=torch.uint8, device=dev)
        self.ws_g = torch.empty(api.quantize_grad_workspace_bytes(L.Cout), **u8)
        self.ws_f = torch.empty(api.conv_workspace_bytes(api.OP_FWD, self.geom), **u8)
        self.ws_d = torch.empty(api.conv_workspace_bytes(api.OP_BWD_DATA, self.geom), **u8)
        self.ws_w = torch.empty(api.conv_workspace_bytes(api.OP_BWD_FILTER, self.geom), **u8)
        self.h_Y = torch.empty(self.Y.shape, dtype=bf).pin_memory()
        self.h_dX = torch.empty(self.dX.shape, dtype=bf).pin_memory()
        self.h_dW = torch.empty(self.dW.shape, dtype=torch.float32).pin_memory()
        self.has_prev = False
        self.h2d = sum(t.numel() * t.element_size() for t in (self.h_x, self.h_w, self.h_g))
        self.d2h = sum(t.numel() * t.element_size() for t in (self.h_Y, self.h_dX, self.h_dW))
        npix_in, npix_out = N * L.H * L.W, N * L.P * L.Q
        wbytes = L.Cout * L.R * L.S * Cip
        # algorithmic bytes / ops per call (operands once, outputs once)
        self.alg = {
            "quantize_x": {"bytes": npix_in * L.Cin * 2 + npix_in * Cip},
            "quantize_w": {"bytes": L.Cout * L.Cin * L.R * L.S * 2 + wbytes},
            "conv_fwd": {"bytes": npix_in * Cip + wbytes + npix_out * L.Cout * 2, "ops": 2 * L.macs(N)},
            "quantize_grad": {"bytes": npix_out * L.Cout * 2 + 2 * npix_out * Cop},
            "conv_bwd_filter": {"bytes": npix_in * Cip + npix_out * Cop + L.Cout * L.Cin * L.R * L.S * 4,
                                "ops": 2 * L.macs(N)},
            "conv_bwd_data": {"bytes": npix_out * Cop + wbytes + npix_in * L.Cin * 2, "ops": 2 * L.macs(N)},
        }

    def calls(self, api, seed):
        L, N = self.L, self.N
        return [
            ("quantize_x", lambda: api.quantize_tensor(self.x, api.NHWC, N, L.Cin, L.H, L.W, api.SCALE_ABSMAX,
                                                       self.sX, api.ROUND_NEAREST_EVEN, 0, self.qX)),
            ("quantize_w", lambda: api.quantize_tensor(self.w, api.NCHW, L.Cout, L.Cin, L.R, L.S, api.SCALE_ABSMAX,
                                                       self.sW, api.ROUND_NEAREST_EVEN, 0, self.qW)),
            ("conv_fwd", lambda: api.conv_fwd(self.qX, self.qW, self.sX, self.sW, self.geom, self.Y, api.NHWC,
                                              self.ws_f)),
            ("quantize_grad", lambda: api.quantize_grad(self.g, api.NHWC, N, L.Cout, L.P, L.Q, None, self.s_state,
                                                        self.has_prev, self.gmax, None, None, self.vq, self.gq,
                                                        seed, self.ws_g)),
            ("conv_bwd_filter", lambda: api.conv_bwd_filter(self.qX, self.vq, self.sX, self.s_state, self.geom,
                                                            self.dW, self.ws_w)),
            ("conv_bwd_data", lambda: api.conv_bwd_data(self.gq, self.qW, self.gmax, self.sW, self.geom, self.dX,
                                                        api.NHWC, self.ws_d)),
        ]


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            p = [t.strip() for t in line.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(names, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def run_dai8(args):
    import torch
    from paper_2102_04782_b200 import api, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    api.lib()

    layers = synth.resnet50_conv2x_block()
    bufs = [LayerBuffers(L, BATCH, SEED + i, torch, api, synth, dev) for i, L in enumerate(layers)]
    step_no = [0]

    def step(record=None):
        seed = SEED + step_no[0]
        for b in bufs:
            for name, fn in b.calls(api, seed):
                if record is not None:
                    e0 = torch.cuda.Event(enable_timing=True); e0.record()
                fn()
                if record is not None:
                    e1 = torch.cuda.Event(enable_timing=True); e1.record()
                    record.append((b.L.name, name, e0, e1))
            b.has_prev = True
        step_no[0] += 1

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_ranks(ms):
        return max_over_ranks(ms, dist, dev)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- timed region: K steps, device-timed, nothing but the path's own launches inside ----------
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = api.launch_count()
    barrier()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    barrier()
    total_ms = max_ranks(t0.elapsed_time(t1))
    launches = api.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    # per-call breakdown: a second, shorter pass of the same steps with an event pair around every call
    # (the events cost device time themselves, so this pass is not the one `value` comes from)
    records = []
    for _ in range(min(args.steps, 100)):
        step(records)
    barrier()
    assert api.get_device_status() == api.OK
    ms_per_step = total_ms / args.steps
    ops_step = bwd_ops(layers, BATCH)
    value = aggregate_value(ops_step, ms_per_step, world)

    # ---- end to end: pinned host inputs -> device, results -> pinned host, every step ------------
    # Two complete sets of device buffers alternate, so that the host->device copy of step i+1 and
    # the device->host copy of step i-1 overlap the kernels of step i (three streams, ordered by
    # events).  Every step still copies all of its inputs in and all of its results out.
    bufs2 = [LayerBuffers(L, BATCH, SEED + i, torch, api, synth, dev) for i, L in enumerate(layers)]
    sets = [bufs, bufs2]
    s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    ev_in = [torch.cuda.Event(), torch.cuda.Event()]
    ev_cmp = [torch.cuda.Event(), torch.cuda.Event()]
    ev_out = [torch.cuda.Event(), torch.cuda.Event()]
    issued = [0]

    def e2e_step():
        i = issued[0]; k = i & 1; set_k = sets[k]
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_cmp[k])          # the kernels of step i-2 have read these inputs
            for b in set_k:
                b.x.copy_(b.h_x, non_blocking=True); b.w.copy_(b.h_w, non_blocking=True)
                b.g.copy_(b.h_g, non_blocking=True)
            ev_in[k].record(s_in)
        s_cmp.wait_event(ev_in[k])
        if i >= 2:
            s_cmp.wait_event(ev_out[k])             # the results of step i-2 have left the device
        seed = SEED + step_no[0]
        for b in set_k:
            for _, fn in b.calls(api, seed):
                fn()
            b.has_prev = True
        step_no[0] += 1
        ev_cmp[k].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[k])
            for b in set_k:
                b.h_Y.copy_(b.Y, non_blocking=True); b.h_dX.copy_(b.dX, non_blocking=True)
                b.h_dW.copy_(b.dW, non_blocking=True)
            ev_out[k].record(s_out)
        issued[0] += 1

    for _ in range(3):
        e2e_step()
    barrier()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e2e_steps = min(args.steps, 40)
    e0.record(s_cmp)
    for _ in range(e2e_steps):
        e2e_step()
    s_cmp.wait_stream(s_out)                        # the last results are on the host
    s_cmp.wait_stream(s_in)
    e1.record(s_cmp)
    barrier()
    e2e_ms = max_ranks(e0.elapsed_time(e1)) / e2e_steps
    e2e_value = aggregate_value(ops_step, e2e_ms, world)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- per-call breakdown and roofline of the dominant call -------------------------------------
    peaks = measured_peaks()
    agg = {}
    for lname, cname, a, b_ in records:
        agg.setdefault((lname, cname), []).append(a.elapsed_time(b_))
    alg = {(b.L.name, k): v for b in bufs for k, v in b.alg.items()}
    detail, dominant = [], None
    sustained = total_ms > 1000.0
    int8_peak = INT8_OVER_BF16 * (peaks["bf16_sustained"] if sustained else peaks["bf16_burst"])
    ridge = int8_peak * 1e12 / (peaks["hbm_gbs"] * 1e9)
    for key, times in agg.items():
        ms = sum(times) / len(times)
        a = alg[key]
        ent = {"layer": key[0], "call": key[1], "ms": round(ms, 5), "gbs": round(a["bytes"] / ms / 1e6, 1)}
        if "ops" in a:
            ent["tops"] = round(a["ops"] / ms / 1e9, 2)
            ent["bound"] = "tensor" if a["ops"] / a["bytes"] > ridge else "hbm"
        else:
            ent["bound"] = "hbm"
        detail.append(ent)
        if dominant is None or ms > dominant[0]:
            dominant = (ms, key, ent)
    dms, dkey, dent = dominant
    if dent["bound"] == "tensor":
        achieved, peak, unit = alg[dkey]["ops"] / dms / 1e9, int8_peak, "TOPS"
    else:
        achieved, peak, unit = alg[dkey]["bytes"] / dms / 1e6, peaks["hbm_gbs"], "GB/s"
    roofline = {"bound": dent["bound"], "achieved": round(achieved, 2), "peak": peak, "unit": unit,
                "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC.get(f"{dkey[1]} @ {dkey[0]}"),
                "algorithmic_bytes": alg[dkey]["bytes"],
                "kernel": f"{dkey[1]} @ {dkey[0]}", "peak_source": peaks["source"],
                "peak_kind": ("int8 = 2 x bf16 " + ("sustained" if sustained else "burst")) if unit == "TOPS" else "copy"}
    def phase_ms(names):
        return sum(e["ms"] for e in detail if e["call"] in names)
    conv_bwd_ms = phase_ms(("conv_bwd_filter", "conv_bwd_data"))
    gvq_ms = phase_ms(("quantize_grad",))
    gvq_bytes = sum(b.alg["quantize_grad"]["bytes"] for b in bufs)
    summary = {
        "conv_bwd_tops_calls_only": round(ops_step / conv_bwd_ms / 1e9, 2),
        "conv_bwd_frac_int8_peak": round(ops_step / conv_bwd_ms / 1e9 / int8_peak, 4),
        "gvq_effective_gbs": round(gvq_bytes / gvq_ms / 1e6, 1),
        "gvq_frac_hbm": round(gvq_bytes / gvq_ms / 1e6 / peaks["hbm_gbs"], 4),
        "int8_peak_tops": int8_peak, "hbm_peak_gbs": peaks["hbm_gbs"], "calls": detail,
    }

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cb = 8
        v, dt, cores = time_oracle(cb, 1, 0)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"same three layers at batch {cb} of {BATCH}, one pass, {dt:.1f} s"}

    line = {
        "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": [l.name for l in layers], "batch": BATCH,
                   "outputs": "Y,dX bf16 NHWC; dW fp32", "l2": "inputs larger than L2 (about 0.9 GB touched per step)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": round(e2e_value, 3), "unit": UNIT, "ms_per_step": round(e2e_ms, 3), "steps": e2e_steps,
                "h2d_bytes_per_step": int(sum(b.h2d for b in bufs)),
                "d2h_bytes_per_step": int(sum(b.d2h for b in bufs))},
        "roofline": roofline, "cpu_baseline": cpu, "detail": summary,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# Per-layer report over one of the network configurations (not the contract line: that is
# run_dai8 on the conv2_x block).  `python bench.py --layers resnet50|mobilenetv2|vgg16 [--batch N]`
# prints one JSON object with, per layer, the device time of the gradient quantization and of the
# three convolutions, and totals as TOPS / GB/s against the measured peaks.
# ------------------------------------------------------------------------------------------------
def run_layer_report(args):
    import torch
    from paper_2102_04782_b200 import api, synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    api.lib()
    table = {"resnet50": (synth.resnet50_convs, 64), "mobilenetv2": (synth.mobilenetv2_pointwise, 128),
             "vgg16": (synth.vgg16_convs, 64), "conv2x": (synth.resnet50_conv2x_block, 64)}
    fn, batch = table[args.layers]
    N = args.batch or batch
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    bf = torch.bfloat16
    rows, seen, no_dx, chain = [], {}, [], {}
    tot = {"fwd": [0.0, 0], "bwd_data": [0.0, 0], "bwd_filter": [0.0, 0], "quantize_grad": [0.0, 0]}

    def timed(call, reps=3):
        best = None
        for _ in range(reps + 1):
            flush.zero_()
            torch.cuda._sleep(200000)   # the host enqueues the call meanwhile, as in a pipelined training step
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(); call(); e1.record(); torch.cuda.synchronize()
            t = e0.elapsed_time(e1)
            best = t if best is None else min(best, t)
        return best

    for L in fn():
        key = (L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.pad)
        if key not in seen:
            g = api.ConvGeom(N, L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.stride, L.pad, L.pad)
            Cip, Cop = api.padded_channels(L.Cin), api.padded_channels(L.Cout)
            qX = torch.randint(-127, 128, (N, L.H, L.W, Cip), dtype=torch.int8, device=dev)
            qW = torch.randint(-127, 128, (L.Cout, L.R, L.S, Cip), dtype=torch.int8, device=dev)
            dY = (torch.randn((N, L.P, L.Q, L.Cout), device=dev) * 1e-4).to(bf)
            vq = torch.empty((N, L.P, L.Q, Cop), dtype=torch.int8, device=dev)
            gq = torch.empty_like(vq)
            Y = torch.empty((N, L.P, L.Q, L.Cout), dtype=bf, device=dev)
            dX = torch.empty((N, L.H, L.W, L.Cin), dtype=bf, device=dev)
            dW = torch.empty((L.Cout, L.Cin, L.R, L.S), dtype=torch.float32, device=dev)
            one = torch.ones(1, device=dev); gm = torch.zeros(1, device=dev)
            s_c = torch.zeros(L.Cout, device=dev)
            ws_g = torch.empty(api.quantize_grad_workspace_bytes(L.Cout), dtype=torch.uint8, device=dev)
            ws_f = torch.empty(max(16, api.conv_workspace_bytes(api.OP_FWD, g)), dtype=torch.uint8, device=dev)
            ws_d = torch.empty(max(16, api.conv_workspace_bytes(api.OP_BWD_DATA, g)), dtype=torch.uint8, device=dev)
            ws_w = torch.empty(max(16, api.conv_workspace_bytes(api.OP_BWD_FILTER, g)), dtype=torch.uint8, device=dev)
            t = {
                "quantize_grad": timed(lambda: api.quantize_grad(dY, api.NHWC, N, L.Cout, L.P, L.Q, None, s_c, False, gm,
                                                                 None, None, vq, gq, 1, ws_g)),
                "fwd": timed(lambda: api.conv_fwd(qX, qW, one, one, g, Y, api.NHWC, ws_f)),
                "bwd_filter": timed(lambda: api.conv_bwd_filter(qX, vq, one, s_c, g, dW, ws_w)),
                "bwd_data": timed(lambda: api.conv_bwd_data(gq, qW, gm, one, g, dX, api.NHWC, ws_d)),
            }
            npix_o, npix_i = N * L.P * L.Q, N * L.H * L.W
            seen[key] = (t, 2 * L.macs(N), npix_o * (2 * L.Cout + 2 * Cop))
            # the same calls again, kept for the pipelined pass below (buffers stay alive in the closures)
            chain[key] = {
                "fwd": lambda qX=qX, qW=qW, g=g, Y=Y, ws_f=ws_f: api.conv_fwd(qX, qW, one, one, g, Y, api.NHWC, ws_f),
                "gvq": lambda dY=dY, L=L, s_c=s_c, gm=gm, vq=vq, gq=gq, ws_g=ws_g: api.quantize_grad(
                    dY, api.NHWC, N, L.Cout, L.P, L.Q, None, s_c, False, gm, None, None, vq, gq, 1, ws_g),
                "dw": lambda qX=qX, vq=vq, s_c=s_c, g=g, dW=dW, ws_w=ws_w: api.conv_bwd_filter(qX, vq, one, s_c, g, dW, ws_w),
                "dx": lambda gq=gq, qW=qW, gm=gm, g=g, dX=dX, ws_d=ws_d: api.conv_bwd_data(gq, qW, gm, one, g, dX, api.NHWC, ws_d),
            }
        t, ops, gvq_bytes = seen[key]
        rows.append({"layer": L.name, "shape": f"{L.Cin}->{L.Cout} {L.R}x{L.S}/{L.stride} @{L.H}",
                     "ms": {k: round(v, 4) for k, v in t.items()},
                     "tops": {k: round(ops / t[k] / 1e9, 1) for k in ("fwd", "bwd_data", "bwd_filter")},
                     "gvq_gbs": round(gvq_bytes / t["quantize_grad"] / 1e6, 1)})
        for k in ("fwd", "bwd_data", "bwd_filter"):
            if k == "bwd_data" and L.Cin == 3:
                no_dx.append(L.name)      # the gradient of the input image has no consumer in training
                continue
            tot[k][0] += t[k]; tot[k][1] += ops
        tot["quantize_grad"][0] += t["quantize_grad"]; tot["quantize_grad"][1] += gvq_bytes
    # ---- the whole network back to back on one stream: forward pass in layer order, backward pass in
    # reverse order (gradient quantization, weight gradient, data gradient per layer), no events or
    # flushes inside; a layer's buffers are shared by its repetitions, the network touches several GB
    order = [(L, (L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.pad)) for L in fn()]

    def run_fwd():
        for L, key in order:
            chain[key]["fwd"]()

    def run_bwd():
        for L, key in reversed(order):
            c = chain[key]
            c["gvq"](); c["dw"]()
            if L.Cin != 3:
                c["dx"]()

    def timed_pass(f):
        best, host = None, None
        for _ in range(4):
            flush.zero_()
            torch.cuda._sleep(2000000)
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            h0 = time.perf_counter(); f(); h1 = time.perf_counter()
            e1.record(); torch.cuda.synchronize()
            t = e0.elapsed_time(e1)
            best = t if best is None else min(best, t)
            host = (h1 - h0) * 1e3 if host is None else min(host, (h1 - h0) * 1e3)
        return best, host

    (pipe_fwd, host_fwd), (pipe_bwd, host_bwd) = timed_pass(run_fwd), timed_pass(run_bwd)
    assert api.get_device_status() == api.OK
    int8_peak = INT8_OVER_BF16 * peaks["bf16_burst"]
    bwd_ms = tot["bwd_data"][0] + tot["bwd_filter"][0]
    bwd_ops = tot["bwd_data"][1] + tot["bwd_filter"][1]
    out = {"layers_config": args.layers, "batch": N, "timing": "best of 3 per call, CUDA events on the device; L2 flushed before each call; the call is enqueued while a delay kernel runs, so host launch latency is not in the time",
           "totals": {
               "fwd_ms": round(tot["fwd"][0], 3), "fwd_tops": round(tot["fwd"][1] / tot["fwd"][0] / 1e9, 1),
               "bwd_ms": round(bwd_ms, 3), "bwd_tops": round(bwd_ops / bwd_ms / 1e9, 1),
               "bwd_frac_int8_peak": round(bwd_ops / bwd_ms / 1e9 / int8_peak, 4),
               "gvq_ms": round(tot["quantize_grad"][0], 3),
               "gvq_gbs": round(tot["quantize_grad"][1] / tot["quantize_grad"][0] / 1e6, 1),
               "gvq_frac_hbm": round(tot["quantize_grad"][1] / tot["quantize_grad"][0] / 1e6 / peaks["hbm_gbs"], 4),
               "int8_peak_tops": int8_peak, "hbm_peak_gbs": peaks["hbm_gbs"]},
           "pipelined": {"fwd_ms": round(pipe_fwd, 3), "bwd_ms_gvq_dw_dx": round(pipe_bwd, 3),
                         "host_enqueue_ms": {"fwd": round(host_fwd, 3), "bwd": round(host_bwd, 3)},
                         "note": "all layers back to back on one stream, best of 4, one event pair around the pass; "
                                 "host_enqueue_ms is the time the Python caller needs to enqueue the pass"},
           "bwd_data_not_counted": no_dx,   # layers fed by the image: timed per layer below, left out of the totals
           "layers": rows}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dai8", choices=["dai8", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", default=None, choices=["conv2x", "resnet50", "mobilenetv2", "vgg16"],
                    help="print a per-layer report for a network configuration instead of the benchmark line")
    ap.add_argument("--batch", type=int, default=0)
    args = ap.parse_args()
    if args.layers:
        run_layer_report(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_dai8(args)


if __name__ == "__main__":
    main()
