#!/usr/bin/env python
"""Benchmark of the dai8 hot path on one B200 (or N independent replicas, one per GPU).

Workload of the JSON line: the thirteen 3x3 convolutions of VGG-16 at N=64, 224x224 input, bf16 NHWC
tensors -- the compute-bound configuration.  One step = the whole path for every layer: forward
quantization of X and W and the int8 forward convolution, layer by layer; then, in reverse layer
order, gradient vectorized quantization of dY (statistics, density count, clip update, vq + gq codes)
and the int8 dW and dX convolutions with de-quantizing epilogues.  Inputs are synthetic
(X = ReLU(N(0,1)), He weights, per-channel bell-shaped / long-tailed dY), drawn on the device.

Prints ONE JSON line.  `value` = int8 backward-convolution throughput, 2*MACs(dX+dW) of the step
divided by the time of the WHOLE step (quantization and the forward pass included), in TOPS, summed
over ranks.  `roofline` describes the kernel with the largest share of the step, `detail` holds the
per-call breakdown (a second pass with a CUDA event pair around every call) and the same totals for
the other configurations (ResNet-50 conv2_x block, all 53 ResNet-50 convolutions, the 34 MobileNetV2
pointwise convolutions), `e2e` the same metric with pinned-host inputs and outputs copied inside the
timed region, `cpu_baseline` the CPU oracle on a bounded sample of the workload.
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
SEED = 2024
INT8_OVER_BF16 = 2.0   # nominal dense ratio 4.5 / 2.25 PFLOP/s


def workloads():
    from paper_2102_04782_b200 import synth
    return {
        "vgg16": ("vgg16_13convs_N64_224x224_bf16_nhwc", synth.vgg16_convs, 64),
        "resnet50": ("resnet50_53convs_N64_224x224_bf16_nhwc", synth.resnet50_convs, 64),
        "mobilenetv2": ("mobilenetv2_34pointwise_N128_224x224_bf16_nhwc", synth.mobilenetv2_pointwise, 128),
        "conv2x": ("resnet50_conv2x_bottleneck_N64_56x56_bf16_nhwc", synth.resnet50_conv2x_block, 64),
    }


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
def oracle_layer_step(L, x, w, g):
    """The whole path for one layer with the CPU oracle, as it stands."""
    from oracle import cpu as O
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


def oracle_inputs(layers, batch):
    from paper_2102_04782_b200 import synth
    return [(L,) + synth.layer_inputs(L, batch, SEED + i, bf16=True)[:3] for i, L in enumerate(layers)]


def bwd_ops(layers, batch):
    return sum(2 * 2 * L.macs(batch) for L in layers)   # dX + dW, 2 ops per MAC


def oracle_pass(workload, batch):
    """One pass of the oracle over every layer of the workload at `batch`: (TOPS, seconds, threads)."""
    from oracle import cpu as O
    _, fn, _ = workloads()[workload]
    layers = fn()
    inputs = oracle_inputs(layers, batch)
    t0 = time.perf_counter()
    for L, x, w, g in inputs:
        oracle_layer_step(L, x, w, g)
    dt = time.perf_counter() - t0
    return bwd_ops(layers, batch) / dt / 1e12, dt, O.num_threads()


def run_reference(args):
    """The oracle as the reference arm.  A full step of the workload would take the CPU many minutes,
    so step i is a bounded sample of it: layer (i mod #layers) of the workload at batch 1."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import cpu as O
    name, fn, batch = workloads()[args.workload]
    layers = fn()
    inputs = oracle_inputs(layers, 1)
    n = len(layers)
    for i in range(args.warmup):
        oracle_layer_step(*inputs[i % n])
    ops, t0 = 0, time.perf_counter()
    for i in range(args.steps):
        L, x, w, g = inputs[i % n]
        oracle_layer_step(L, x, w, g)
        ops += bwd_ops([L], 1)
    dt = time.perf_counter() - t0
    value = ops / dt / 1e12
    sample = (f"step i = the whole path for layer (i mod {n}) of the workload at batch 1 of {batch} "
              "(bounded sample), CPU oracle as it stands")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": sample},
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
GRAPH_SEEDS = 4                 # CUDA graphs of the step, one per rounding seed, replayed in turn
BLOCKER_CYCLES = 16_000_000     # about 8 ms of device spin in front of a step of the per-call breakdown


class LayerBuffers:
    """Device buffers of one layer; `host` adds pinned host copies of the inputs and results."""

    def __init__(self, L, N, seed, torch, api, synth, dev, host=None):
        self.L, self.N = L, N
        bf = torch.bfloat16
        self.x, self.w, self.g = synth.device_layer_inputs(L, N, seed, dev)
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
        self.cls = torch.zeros(L.Cout, dtype=torch.uint8, device=dev)
        self.Y = torch.empty((N, L.P, L.Q, L.Cout), dtype=bf, device=dev)
        self.dX = torch.empty((N, L.H, L.W, L.Cin), dtype=bf, device=dev)
        self.dW = torch.empty((L.Cout, L.Cin, L.R, L.S), **f32)
        u8 = dict(dtype=torch.uint8, device=dev)
        self.ws_q = torch.empty(max(16, api.quantize_tensor_workspace_bytes()), **u8)
        self.ws_g = torch.empty(api.quantize_grad_workspace_bytes(L.Cout), **u8)
        self.ws_f = torch.empty(max(16, api.conv_workspace_bytes(api.OP_FWD, self.geom)), **u8)
        self.ws_d = torch.empty(max(16, api.conv_workspace_bytes(api.OP_BWD_DATA, self.geom)), **u8)
        self.ws_w = torch.empty(max(16, api.conv_workspace_bytes(api.OP_BWD_FILTER, self.geom)), **u8)
        self.has_prev = False
        self.host = host
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

    def fwd_calls(self, api):
        L, N = self.L, self.N
        return [
            ("quantize_x", lambda: api.quantize_tensor(self.x, api.NHWC, N, L.Cin, L.H, L.W, api.SCALE_ABSMAX,
                                                       self.sX, api.ROUND_NEAREST_EVEN, 0, self.qX, self.ws_q)),
            ("quantize_w", lambda: api.quantize_tensor(self.w, api.NCHW, L.Cout, L.Cin, L.R, L.S, api.SCALE_ABSMAX,
                                                       self.sW, api.ROUND_NEAREST_EVEN, 0, self.qW, self.ws_q)),
            ("conv_fwd", lambda: api.conv_fwd(self.qX, self.qW, self.sX, self.sW, self.geom, self.Y, api.NHWC,
                                              self.ws_f)),
        ]

    def bwd_calls(self, api, seed):
        L, N = self.L, self.N
        return [
            ("quantize_grad", lambda: api.quantize_grad(self.g, api.NHWC, N, L.Cout, L.P, L.Q, None, self.s_state,
                                                        self.has_prev, self.gmax, None, self.cls, self.vq, self.gq,
                                                        seed, self.ws_g)),
            ("conv_bwd_filter", lambda: api.conv_bwd_filter(self.qX, self.vq, self.sX, self.s_state, self.geom,
                                                            self.dW, self.ws_w)),
            ("conv_bwd_data", lambda: api.conv_bwd_data(self.gq, self.qW, self.gmax, self.sW, self.geom, self.dX,
                                                        api.NHWC, self.ws_d)),
        ]


class HostBuffers:
    """Pinned host copies of one layer's inputs (X, W, dY) and room for its results (Y, dX, dW)."""

    def __init__(self, b, torch):
        self.x, self.w, self.g = (t.cpu().pin_memory() for t in (b.x, b.w, b.g))
        self.Y = torch.empty(b.Y.shape, dtype=b.Y.dtype).pin_memory()
        self.dX = torch.empty(b.dX.shape, dtype=b.dX.dtype).pin_memory()
        self.dW = torch.empty(b.dW.shape, dtype=b.dW.dtype).pin_memory()
        self.h2d = sum(t.numel() * t.element_size() for t in (self.x, self.w, self.g))
        self.d2h = sum(t.numel() * t.element_size() for t in (self.Y, self.dX, self.dW))


class ClockSampler:
    """nvidia-smi in a loop, started before the warm-up; stop() keeps the samples whose time stamps
    fall between mark_start() and mark_end() (all of them if too few do)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc, self.t0, self.t1 = None, None, None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        import datetime
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            p = [t.strip() for t in line.split(",")]
            if len(p) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(p[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(p[1]), float(p[2]), float(p[3]),
                             [n for n, v in zip(names, p[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in rows if self.t0 is not None and self.t0 - 0.02 <= r[0] <= self.t1 + 0.02]
        window = "timed region"
        if len(inside) < 3:      # a very short timed region: the loaded samples of the whole run instead
            busy = [r for r in rows if r[3] > 250.0]
            inside, window = (busy if len(busy) >= 3 else rows), "whole run (timed region too short to sample)"
        sm = [r[1] for r in inside]
        reasons = sorted({n for r in inside for n in r[4]})
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max((r[2] for r in inside), default=None),
                "power_w_max": max((r[3] for r in inside), default=None),
                "samples": len(inside), "window": window, "reasons": reasons}


class Runner:
    """One workload on one GPU: buffers, the step, the timed region, the per-call breakdown."""

    def __init__(self, workload, torch, api, synth, dev, dist, world, with_host=False, batch=0):
        self.torch, self.api, self.dev, self.dist, self.world = torch, api, dev, dist, world
        self.name, fn, self.batch = workloads()[workload]
        if batch:                       # a reduced batch, for profiler captures of a small case
            self.batch = batch
            self.name += f"_batch{batch}"
        self.layers = fn()
        self.bufs = [LayerBuffers(L, self.batch, SEED + i, torch, api, synth, dev) for i, L in enumerate(self.layers)]
        self.step_no = 0
        self.kernel_of = {}             # (layer, call) -> kernel family, as the library reports it
        self.ops_step = bwd_ops(self.layers, self.batch)
        self.hosts = [HostBuffers(b, torch) for b in self.bufs] if with_host else None

    def step(self, bufs=None, record=None):
        torch, api = self.torch, self.api
        bufs = bufs or self.bufs
        seed = SEED + self.step_no

        def run(b, calls):
            for name, fn in calls:
                if record is not None:
                    e0 = torch.cuda.Event(enable_timing=True); e0.record()
                fn()
                if record is not None:
                    e1 = torch.cuda.Event(enable_timing=True); e1.record()
                    record.append((b.L.name, name, e0, e1))
                    self.kernel_of[(b.L.name, name)] = api.debug_last_kernel()

        for b in bufs:                      # forward pass, layer order
            run(b, b.fwd_calls(api))
        for b in reversed(bufs):            # backward pass, reverse order
            run(b, b.bwd_calls(api, seed))
            b.has_prev = True
        self.step_no += 1

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def capture(self, n_graphs=GRAPH_SEEDS):
        """The step as CUDA graphs: every entry point only enqueues work on the stream it is given
        (no allocation, no synchronisation), so a whole step is captured once and replayed.  The seed of
        the stochastic rounding is a by-value argument, hence one graph per seed; the replays cycle
        through n_graphs of them.  Returns the kernel launches of one step."""
        torch, api = self.torch, self.api
        self.graphs = []
        per_step = 0
        for _ in range(n_graphs):
            g = torch.cuda.CUDAGraph()
            n0 = api.launch_count()
            with torch.cuda.graph(g):
                self.step()
            per_step = api.launch_count() - n0
            self.graphs.append(g)
        self.barrier()
        return per_step

    def timed(self, steps, warmup, sampler=None, graph=True):
        torch, api = self.torch, self.api
        for _ in range(max(warmup, 3)):     # eager: first-use initialisation happens outside any capture
            self.step()
        self.barrier()
        per_step = self.capture() if graph else 0
        if graph:
            for i in range(max(warmup, 3)):
                self.graphs[i % len(self.graphs)].replay()
            self.barrier()
        launches0 = api.launch_count()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        if sampler:
            sampler.mark_start()
        t0.record()
        for i in range(steps):
            if graph:
                self.graphs[i % len(self.graphs)].replay()
            else:
                self.step()
        t1.record()
        self.barrier()
        if sampler:
            sampler.mark_end()
        total_ms = max_over_ranks(t0.elapsed_time(t1), self.dist, self.dev)
        launches = per_step * steps if graph else api.launch_count() - launches0
        assert api.get_device_status() == api.OK
        self.graphs = []
        return total_ms, launches

    def breakdown(self, steps):
        """Second pass with a CUDA event pair around every call (the events keep consecutive kernels
        from overlapping, so this pass is not the one `value` comes from)."""
        records = []
        for _ in range(steps):
            # the host enqueues a step of small layers more slowly than the GPU runs it; a spin of a few
            # milliseconds in front lets the host get ahead, so the event pairs bracket device time only
            self.torch.cuda._sleep(BLOCKER_CYCLES)
            self.step(record=records)
            self.torch.cuda.synchronize()
        self.barrier()
        agg = {}
        for lname, cname, a, b_ in records:
            agg.setdefault((lname, cname), []).append(a.elapsed_time(b_))
        return {k: sum(v) / len(v) for k, v in agg.items()}

    def e2e(self, steps):
        """Pinned host inputs -> device, results -> pinned host, every step.  Two complete sets of device
        buffers alternate, so that the host->device copy of step i+1 and the device->host copy of step
        i-1 overlap the kernels of step i (three streams, ordered by events).  Every step still copies
        all of its inputs in and all of its results out."""
        torch, api = self.torch, self.api
        from paper_2102_04782_b200 import synth
        bufs2 = [LayerBuffers(L, self.batch, SEED + i, torch, api, synth, self.dev) for i, L in enumerate(self.layers)]
        sets = [self.bufs, bufs2]
        hosts = self.hosts
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
                for b, h in zip(set_k, hosts):
                    b.x.copy_(h.x, non_blocking=True); b.w.copy_(h.w, non_blocking=True)
                    b.g.copy_(h.g, non_blocking=True)
                ev_in[k].record(s_in)
            s_cmp.wait_event(ev_in[k])
            if i >= 2:
                s_cmp.wait_event(ev_out[k])             # the results of step i-2 have left the device
            self.step(bufs=set_k)
            ev_cmp[k].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[k])
                for b, h in zip(set_k, hosts):
                    h.Y.copy_(b.Y, non_blocking=True); h.dX.copy_(b.dX, non_blocking=True)
                    h.dW.copy_(b.dW, non_blocking=True)
                ev_out[k].record(s_out)
            issued[0] += 1

        for _ in range(3):
            e2e_step()
        self.barrier()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(s_cmp)
        for _ in range(steps):
            e2e_step()
        s_cmp.wait_stream(s_out)                        # the last results are on the host
        s_cmp.wait_stream(s_in)
        e1.record(s_cmp)
        self.barrier()
        ms = max_over_ranks(e0.elapsed_time(e1), self.dist, self.dev) / steps
        return ms, int(sum(h.h2d for h in hosts)), int(sum(h.d2h for h in hosts))

    def summarize(self, per_call_ms, int8_peak, peaks):
        """Per-call entries, phase totals and the dominant kernel of the step."""
        alg = {(b.L.name, k): v for b in self.bufs for k, v in b.alg.items()}
        shape = {b.L.name: f"{b.L.Cin}->{b.L.Cout} {b.L.R}x{b.L.S}/{b.L.stride} @{b.L.H}" for b in self.bufs}
        ridge = int8_peak * 1e12 / (peaks["hbm_gbs"] * 1e9)
        calls, by_call = [], {}
        for key, ms in per_call_ms.items():
            a = alg[key]
            ent = {"layer": key[0], "shape": shape[key[0]], "call": key[1], "ms": round(ms, 5),
                   "gbs": round(a["bytes"] / ms / 1e6, 1)}
            if "ops" in a:
                ent["tops"] = round(a["ops"] / ms / 1e9, 1)
                ent["frac_int8_peak"] = round(a["ops"] / ms / 1e9 / int8_peak, 4)
                ent["bound"] = "tensor" if a["ops"] / a["bytes"] > ridge else "hbm"
            else:
                ent["frac_hbm"] = round(a["bytes"] / ms / 1e6 / peaks["hbm_gbs"], 4)
                ent["bound"] = "hbm"
            calls.append(ent)
            t = by_call.setdefault(key[1], {"ms": 0.0, "bytes": 0, "ops": 0, "n": 0, "tensor_ms": 0.0, "tensor_ops": 0})
            t["ms"] += ms; t["bytes"] += a["bytes"]; t["ops"] += a.get("ops", 0); t["n"] += 1
            if ent["bound"] == "tensor":
                t["tensor_ms"] += ms; t["tensor_ops"] += a["ops"]
        total = sum(t["ms"] for t in by_call.values())
        phases = {}
        for name, t in by_call.items():
            p = {"ms": round(t["ms"], 4), "share": round(t["ms"] / total, 4), "launch_groups": t["n"],
                 "gbs": round(t["bytes"] / t["ms"] / 1e6, 1), "frac_hbm": round(t["bytes"] / t["ms"] / 1e6 / peaks["hbm_gbs"], 4)}
            if t["ops"]:
                p["tops"] = round(t["ops"] / t["ms"] / 1e9, 1)
                p["frac_int8_peak"] = round(t["ops"] / t["ms"] / 1e9 / int8_peak, 4)
            if t["tensor_ms"] > 0:
                p["compute_bound_layers_tops"] = round(t["tensor_ops"] / t["tensor_ms"] / 1e9, 1)
                p["compute_bound_layers_frac_int8_peak"] = round(t["tensor_ops"] / t["tensor_ms"] / 1e9 / int8_peak, 4)
            phases[name] = p
        bwd = [by_call.get("conv_bwd_filter"), by_call.get("conv_bwd_data")]
        bwd_ms = sum(t["ms"] for t in bwd if t)
        bwd_ops_ = sum(t["ops"] for t in bwd if t)
        gvq = by_call.get("quantize_grad")
        out = {"phases": phases,
               "conv_bwd_tops_calls_only": round(bwd_ops_ / bwd_ms / 1e9, 1),
               "conv_bwd_frac_int8_peak": round(bwd_ops_ / bwd_ms / 1e9 / int8_peak, 4),
               "gvq_effective_gbs": round(gvq["bytes"] / gvq["ms"] / 1e6, 1),
               "gvq_frac_hbm": round(gvq["bytes"] / gvq["ms"] / 1e6 / peaks["hbm_gbs"], 4)}
        # the same calls grouped by the kernel that served them: the dominant KERNEL of the step
        by_kernel = {}
        for key, ms in per_call_ms.items():
            a = alg[key]
            t = by_kernel.setdefault(self.kernel_of.get(key, key[1]), {"ms": 0.0, "bytes": 0, "ops": 0, "n": 0, "calls": set()})
            t["ms"] += ms; t["bytes"] += a["bytes"]; t["ops"] += a.get("ops", 0); t["n"] += 1; t["calls"].add(key[1])
        kernels = {}
        for name, t in sorted(by_kernel.items(), key=lambda kv: -kv[1]["ms"]):
            k = {"ms": round(t["ms"], 4), "share": round(t["ms"] / total, 4), "launch_groups": t["n"],
                 "calls": sorted(t["calls"]), "gbs": round(t["bytes"] / t["ms"] / 1e6, 1),
                 "frac_hbm": round(t["bytes"] / t["ms"] / 1e6 / peaks["hbm_gbs"], 4)}
            if t["ops"]:
                k["tops"] = round(t["ops"] / t["ms"] / 1e9, 1)
                k["frac_int8_peak"] = round(t["ops"] / t["ms"] / 1e9 / int8_peak, 4)
            kernels[name] = k
        out["kernels"] = kernels
        dom_name = max(by_kernel, key=lambda n: by_kernel[n]["ms"])
        return out, calls, dom_name, by_kernel[dom_name]


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
    peaks = measured_peaks()

    sampler = ClockSampler(local) if rank == 0 else None
    main = Runner(args.workload, torch, api, synth, dev, dist, world, with_host=True, batch=args.batch)
    warmup = max(args.warmup, 3)
    total_ms, launches = main.timed(args.steps, warmup, sampler, graph=not args.eager)
    clocks = sampler.stop() if sampler else None
    ms_per_step = total_ms / args.steps
    value = aggregate_value(main.ops_step, ms_per_step, world)
    sustained = total_ms > 1000.0
    int8_peak = INT8_OVER_BF16 * (peaks["bf16_sustained"] if sustained else peaks["bf16_burst"])
    per_call = main.breakdown(min(args.steps, 10))
    e2e_steps = max(2, min(args.steps, 8))
    e2e_ms, h2d, d2h = main.e2e(e2e_steps)
    e2e_value = aggregate_value(main.ops_step, e2e_ms, world)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    summary, calls, dom_name, dom = main.summarize(per_call, int8_peak, peaks)
    tensor_bound = dom["ops"] > 0 and dom["ops"] / dom["bytes"] > int8_peak * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if tensor_bound:
        achieved, peak, unit = dom["ops"] / dom["ms"] / 1e9, int8_peak, "TOPS"
    else:
        achieved, peak, unit = dom["bytes"] / dom["ms"] / 1e6, peaks["hbm_gbs"], "GB/s"
    roofline = {"bound": "tensor" if tensor_bound else "hbm", "achieved": round(achieved, 2), "peak": peak,
                "unit": unit, "frac": round(achieved / peak, 4), "traffic": None,
                "kernel": dom_name, "launches_per_step": dom["n"], "calls": sorted(dom["calls"]),
                "share_of_step": summary["kernels"][dom_name]["share"],
                "algorithmic_ops_per_step": dom["ops"], "algorithmic_bytes_per_step": dom["bytes"],
                "ms_per_step": round(dom["ms"], 4), "peak_source": peaks["source"],
                "peak_kind": ("int8 = 2 x bf16 " + ("sustained" if sustained else "burst")) if unit == "TOPS" else "copy",
                "note": "all launches of this kernel in one step, summed: achieved = their algorithmic ops (bytes) / their time"}
    summary["calls"] = calls
    summary["int8_peak_tops"] = int8_peak
    summary["hbm_peak_gbs"] = peaks["hbm_gbs"]
    summary["targets"] = {"conv_bwd_frac_int8_peak_on_compute_bound_layers": 0.60, "gvq_frac_hbm": 0.70}
    del main
    torch.cuda.empty_cache()

    # ---- the other configurations, device-timed the same way (no end-to-end leg) -------------------
    others = {}
    if world == 1 and not args.main_only:
        for wl in ("conv2x", "resnet50", "mobilenetv2", "vgg16"):
            if wl == args.workload:
                continue
            r = Runner(wl, torch, api, synth, dev, None, 1)
            steps = min(args.steps, 20)
            t_ms, _ = r.timed(steps, 3, graph=not args.eager)
            s, c, _, _ = r.summarize(r.breakdown(min(steps, 5)), INT8_OVER_BF16 * peaks["bf16_burst"], peaks)
            s["workload"] = r.name
            s["ms_per_step"] = round(t_ms / steps, 4)
            s["value_tops"] = round(aggregate_value(r.ops_step, t_ms / steps, 1), 2)
            s["compute_bound_calls"] = [e for e in c if e["bound"] == "tensor"]
            others[wl] = s
            del r
            torch.cuda.empty_cache()
    summary["other_configs"] = others

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, dt, cores = oracle_pass(args.workload, 1)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"every layer of the workload at batch 1 of {workloads()[args.workload][2]}, one pass, {dt:.1f} s"}

    name, _, batch = workloads()[args.workload]
    line = {
        "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": name, "layers": len(workloads()[args.workload][1]()), "batch": batch,
                   "outputs": "Y,dX bf16 NHWC; dW fp32",
                   "l2": "inputs larger than L2 (several GB touched per step)",
                   "launch": "eager, one library call after another" if args.eager else
                             f"the step captured in CUDA graphs (one per rounding seed, {GRAPH_SEEDS} seeds in turn) and replayed",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": round(e2e_value, 3), "unit": UNIT, "ms_per_step": round(e2e_ms, 3), "steps": e2e_steps,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "roofline": roofline, "cpu_baseline": cpu, "detail": summary,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# Per-layer report over one of the network configurations (not the contract line).
# `python bench.py --layers resnet50|mobilenetv2|vgg16|conv2x [--batch N]` prints one JSON object
# with, per layer, the device time of the gradient quantization and of the three convolutions in
# isolation (L2 flushed, best of 3), and the whole network back to back with the host enqueue time.
# ------------------------------------------------------------------------------------------------
def run_layer_report(args):
    import torch
    from paper_2102_04782_b200 import api, synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    api.lib()
    _, fn, batch = workloads()[args.layers]
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
            npix_o = N * L.P * L.Q
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
    bwd_ops_ = tot["bwd_data"][1] + tot["bwd_filter"][1]
    out = {"layers_config": args.layers, "batch": N, "timing": "best of 3 per call, CUDA events on the device; L2 flushed before each call; the call is enqueued while a delay kernel runs, so host launch latency is not in the time",
           "totals": {
               "fwd_ms": round(tot["fwd"][0], 3), "fwd_tops": round(tot["fwd"][1] / tot["fwd"][0] / 1e9, 1),
               "bwd_ms": round(bwd_ms, 3), "bwd_tops": round(bwd_ops_ / bwd_ms / 1e9, 1),
               "bwd_frac_int8_peak": round(bwd_ops_ / bwd_ms / 1e9 / int8_peak, 4),
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


def run_probe(args):
    """The two micro-measurements the kernel designs lean on, from the library's own debug entries."""
    import torch
    from paper_2102_04782_b200 import api
    torch.cuda.set_device(0)
    api.lib()
    ws = torch.empty(64, dtype=torch.uint8, device="cuda")
    peaks = measured_peaks()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    mhz = 1965.0
    mma = []
    for rb in (128, 64, 32):
        for n in (16, 64, 128, 256):
            issue, done = api.debug_probe_mma(n, rb, 4096, ws)
            mma.append({"n_cols": n, "row_bytes": rb, "issue_cycles": round(issue, 1), "complete_cycles": round(done, 1),
                        "tops_at_max_clock": round(2 * 128 * n * 32 / done * mhz * 1e6 * sms / 1e12, 1)})
    sr = api.debug_probe_sr(2000, ws)
    out = {"probe": "tcgen05.mma.kind::i8 issue rate and stochastic-rounding arithmetic rate", "sms": sms,
           "sm_max_mhz_assumed": mhz, "mma_m128_k32": mma,
           "sr_elements_per_second": sr, "sr_equivalent_gbs_bf16_dual": round(sr * 4 / 1e9, 1),
           "note": "tops_at_max_clock = 2*128*N*32 / complete_cycles * clock * SMs; sr_equivalent_gbs = elements/s x (2 B in + 2 B out)",
           "int8_proxy_peak_tops": INT8_OVER_BF16 * peaks["bf16_burst"], "hbm_peak_gbs": peaks["hbm_gbs"]}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dai8", choices=["dai8", "reference"])
    ap.add_argument("--workload", default="vgg16", choices=["vgg16", "resnet50", "mobilenetv2", "conv2x"],
                    help="configuration of the JSON line (default: VGG-16, the compute-bound one)")
    ap.add_argument("--main-only", action="store_true", help="skip the other configurations in `detail`")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true", help="time eager library calls instead of CUDA-graph replays of the step")
    ap.add_argument("--layers", default=None, choices=["conv2x", "resnet50", "mobilenetv2", "vgg16"],
                    help="print a per-layer report for a network configuration instead of the benchmark line")
    ap.add_argument("--batch", type=int, default=0, help="reduced batch (profiler captures of a small case; not a benchmark result)")
    ap.add_argument("--probe", action="store_true", help="print the tcgen05.mma issue-rate and rounding-arithmetic micro-measurements")
    args = ap.parse_args()
    if args.probe:
        run_probe(args)
    elif args.layers:
        run_layer_report(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_dai8(args)


if __name__ == "__main__":
    main()
