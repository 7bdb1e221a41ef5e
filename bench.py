#!/usr/bin/env python
"""Throughput of the channel-gated convolution layers on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload cifar|imagenet] [--density D] [--rho R] [--cond-mode M]

One step = one forward pass of every gated 3x3 layer shape of the workload over one batch
of synthetic activations (ReLU of box-smoothed Gaussian noise, bf16).  Prints ONE JSON line:
the headline value on --workload, every layer at the target density and with all gates open
(`speedup_vs_density1` against `flop_reduction`), and, at one GPU, extra blocks for the ImageNet
shapes, G = 8, a density sweep, cross-channel correlated inputs and the int8 layers.
Under torchrun each rank runs the same layers on its own batch (weak scaling, no collective
on the data path); the time is the max over ranks.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "gated-conv images/sec at measured gate density"
UNIT = "images/s"


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the layer kernel:
# the mean over the six launches listed in profiles/dram_traffic_layer_kernels.txt.  The y and mask
# writes of a captured launch are still in the 126 MB L2 when it ends, so they are not in these
# sums.  Reported only while the kernel sources still hash to what they were when the counters
# were taken.
KERNEL_NAMES = ["direct", "tcgen05 pixel-major", "tcgen05 channel-major", "tcgen05 tap-stacked"]

TRAFFIC = {
    "source_sha": "25f6222633311712",
    "bytes_per_launch": {"c64@32": 33790250, "c128@16": 17143296, "c256@8": 9645397, "c512@4": 9110314},
}


def kernel_source_sha():
    import glob
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1805_12549_b200", "csrc")
    for path in sorted(glob.glob(os.path.join(csrc, "*.cu")) + glob.glob(os.path.join(csrc, "*.cuh"))):
        h.update(open(path, "rb").read())
    return h.hexdigest()[:16]


def measured_traffic(layer_name):
    if TRAFFIC["source_sha"] != kernel_source_sha():
        return None
    return TRAFFIC["bytes_per_launch"].get(layer_name)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def workload_layers(name, batch=None):
    from paper_1805_12549_b200 import synth
    if name == "cifar":
        return "cifar_resnet18_gated_3x3_layers", synth.cifar_resnet18_layers(batch or 256, 4)
    if name == "imagenet":
        return "imagenet_resnet18_gated_3x3_layers", synth.imagenet_resnet18_layers(batch or 64, 4)
    raise SystemExit(f"unknown workload {name}")


# ------------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms",
                 "100", "-i", str(index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for t, line in self.samples:
            if t < t0 - 0.05 or t > t1 + 0.15:
                continue
            f = [v.strip() for v in line.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------- ranks
def max_over_ranks(ms_local, device="cuda"):
    """Device time of the slowest rank (every rank shards the batch and runs alone: no
    collective on the data path, only this reduction of the timing)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(images_per_rank, world, ms_per_step):
    """Aggregate images/s of `world` ranks that each process `images_per_rank` per step."""
    return world * images_per_rank / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------- our arm
CALIB_IMAGES = 4     # gate statistics and Delta come from the first images of the batch (both arms)


def calibrate(p, density, eps=1e-5):
    """Gate statistics = per-channel mean/variance of the partial sums `p` [pixels, c_out] (what a
    trained network's running statistics would hold); Delta = one scalar per layer at the quantile
    of the normalised partial sums that gives the target density.  Used by both arms, on the
    partial sums of the first CALIB_IMAGES images."""
    p = np.asarray(p, np.float64)
    mean = p.mean(0).astype(np.float32)
    var = np.maximum(p.var(0), 1e-6).astype(np.float32)
    p_hat = (p - mean) / np.sqrt(var.astype(np.float64) + eps)
    return mean, var, p_hat.ravel()


def delta_for(p_hat, density):
    if density >= 1.0:
        return float("-inf")
    if density <= 0.0:
        return float("inf")
    return float(np.quantile(p_hat, 1.0 - density))


class LayerBench:
    """Device buffers, calibrated gate parameters and the handle of one layer shape."""

    SETS = 4   # x/y/mask buffer sets rotated so that no step finds its tensors in L2

    def __init__(self, shape, rho, cond_mode, rank, dtype="bf16", host=False):
        import torch
        from paper_1805_12549_b200 import binding as B, synth
        self.B, self.torch, self.shape, self.dtype = B, torch, shape, dtype
        s = shape
        key = ("bench", s.name, rank)
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
        calib = min(CALIB_IMAGES, s.n)
        if dtype == "bf16":
            x = synth.bf16_bits(synth.smoothed_noise((key, "x"), s.n, s.hw, s.hw, s.c_in, rho=rho))
            wb, wc = synth.kaiming_weights(key, s.c_out, 3, 3, s.c_in, s.groups)
            bf = lambda a: dev(synth.bf16_bits(a).view(np.int16)).view(torch.bfloat16)
            x0 = dev(x.view(np.int16)).view(torch.bfloat16)
            self.wb, self.wc = bf(wb), bf(wc)
            self.conv = B.GatedConv(s.n, s.hw, s.hw, s.c_in, s.c_out, k=3, stride=s.stride, pad=1,
                                    groups=s.groups, dtype=B.CG_BF16, cond_mode=cond_mode)
            self.params = {k: dev(v) for k, v in synth.bn_params(key, s.c_out).items()}
            cal = B.GatedConv(calib, s.hw, s.hw, s.c_in, s.c_out, k=3, stride=s.stride, pad=1,
                              groups=s.groups, dtype=B.CG_BF16, algo=B.CG_ALGO_DIRECT)
            p = torch.empty((cal.m, s.c_out), dtype=torch.float32, device="cuda")
            B.cg_conv_partial_sums(cal.handle, x0[:calib].contiguous(), self.wb, p)
            torch.cuda.synchronize()
            mean, var, self.p_hat = calibrate(p.cpu().numpy(), None)
            cal.close()
            self.params["gate_mean"], self.params["gate_var"] = dev(mean), dev(var)
            self.delta = torch.zeros((s.c_out,), dtype=torch.float32, device="cuda")
            el = 2
        else:
            x0 = dev(synth.int8_activations(key, s.n, s.hw, s.hw, s.c_in))
            wb, wc = synth.int8_weights(key, s.c_out, 3, 3, s.c_in, s.groups)
            self.wb, self.wc = dev(wb), dev(wc)
            self.conv = B.GatedConv(s.n, s.hw, s.hw, s.c_in, s.c_out, k=3, stride=s.stride, pad=1,
                                    groups=s.groups, dtype=B.CG_I8, requant_shift=24, cond_mode=cond_mode)
            cal = B.GatedConv(calib, s.hw, s.hw, s.c_in, s.c_out, k=3, stride=s.stride, pad=1,
                              groups=s.groups, dtype=B.CG_I8, requant_shift=24, algo=B.CG_ALGO_DIRECT)
            p = torch.empty((cal.m, s.c_out), dtype=torch.int32, device="cuda")
            B.cg_conv_partial_sums(cal.handle, x0[:calib].contiguous(), self.wb, p)
            torch.cuda.synchronize()
            self.p_int = p.cpu().numpy().astype(np.float64)
            cal.close()
            sigma_base = self.p_int.std() + 1.0
            q = synth.int8_requant(key, s.c_out, 24, sigma_base, sigma_base * np.sqrt(s.groups))
            self.params = {k: dev(v) for k, v in q.items()}
            self.params["q_gate_thr"] = torch.zeros((s.c_out,), dtype=torch.int32, device="cuda")
            self.delta = None
            el = 1
        self.xs = [x0] + [torch.roll(x0, k, dims=0).contiguous() for k in range(1, self.SETS)]
        self.bn = B.make_bn(self.params)
        self.ys, self.masks = zip(*[self.conv.alloc_outputs() for _ in range(self.SETS)])
        if host:
            self.x_host = x0.cpu().pin_memory()
            self.y_host = torch.empty(self.ys[0].shape, dtype=self.ys[0].dtype).pin_memory()
            self.mask_host = torch.empty(self.masks[0].shape, dtype=torch.int32).pin_memory()
            self.staging = torch.empty(B.cg_conv_host_staging_bytes(self.conv.handle),
                                       dtype=torch.uint8, device="cuda")
        self.bytes_x = s.n * s.hw * s.hw * s.c_in * el
        self.bytes_y = self.conv.m * s.c_out * el
        self.bytes_mask = self.conv.m * self.conv.words * 4
        self.bytes_w = s.c_out * 9 * s.c_in * el
        self.algorithmic_bytes = self.bytes_x + self.bytes_y + self.bytes_mask + self.bytes_w
        self.stats = None

    def set_density(self, density):
        """Rewrites Delta (or the integer thresholds) in place: captured graphs read the new values."""
        if self.dtype == "bf16":
            self.delta.fill_(delta_for(self.p_hat, density))
        else:
            if density >= 1.0:
                thr = np.full(self.shape.c_out, np.iinfo(np.int32).min, np.int64)
            else:
                thr = np.ceil(np.quantile(self.p_int, 1.0 - density, axis=0))
            self.params["q_gate_thr"].copy_(self.torch.from_numpy(thr.astype(np.int32)))

    def forward(self, i):
        k = i % self.SETS
        self.conv.forward(self.xs[k], self.wb, self.wc, self.bn, self.delta, self.ys[k],
                          self.masks[k])

    def forward_host(self, stream=None):
        self.B.cg_conv_forward_host(self.conv.handle, self.x_host, self.wb, self.wc, self.bn,
                                    self.delta, None, self.y_host, self.mask_host, self.staging, stream)

    def close(self):
        self.conv.close()


class Plain:
    def __init__(self, fn):
        self.fn = fn

    def replay(self):
        self.fn()


def capture(fn, no_graph):
    """Launches go through CUDA graphs (one graph = the captured calls on fixed buffer sets), so
    the device, not the Python caller, sets the pace."""
    import torch
    if no_graph:
        return Plain(fn)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def time_layer(lb, reps, no_graph):
    """Average device time of one launch of the layer kernel (CUDA events on the launching
    stream), the buffer sets rotating so that no launch finds its tensors in L2."""
    import torch
    stream = torch.cuda.current_stream()
    g = capture(lambda: [lb.forward(k) for k in range(LayerBench.SETS)], no_graph)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g.replay()
    torch.cuda.synchronize()
    lb.conv.stats()
    e0.record(stream)
    for _ in range(reps):
        g.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    st = lb.conv.stats()
    return e0.elapsed_time(e1) / (reps * LayerBench.SETS), st


def layer_record(lb, d_ms, st, peaks):
    el_flops = 2.0 * st.gated_macs / max(st.calls, 1)
    t_tensor = el_flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = lb.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9)
    rec = {
        "layer": lb.shape.name, "us": round(d_ms * 1e3, 2), "density": round(st.density, 4),
        "kernel": KERNEL_NAMES[lb.conv.kernel_id],
        "gated_tflops": round(el_flops / (d_ms * 1e-3) / 1e12, 1),
        "gbs": round(lb.algorithmic_bytes / (d_ms * 1e-3) / 1e9, 1),
        "roof_us": round(max(t_tensor, t_hbm) * 1e6, 2),
        "roof_frac": round(max(t_tensor, t_hbm) / (d_ms * 1e-3), 3),
        "bound": "tensor" if t_tensor > t_hbm else "hbm",
        "flop_reduction": round(st.dense_macs / max(st.gated_macs, 1), 3),
        "executed_over_gated": round(st.executed_macs / max(st.gated_macs, 1), 3),
        "blocks_skipped": f"{st.tiles_skipped}/{st.tiles_total}",
    }
    if lb.dtype != "bf16":
        # no measured int8 tensor peak on this machine: the fraction is against the HBM side only
        rec["roof_us"] = round(t_hbm * 1e6, 2)
        rec["roof_frac"] = round(t_hbm / (d_ms * 1e-3), 3)
        rec["bound"] = "hbm (no int8 tensor peak measured)"
    return rec


def with_density1(lb, rec, reps, no_graph, peaks, target):
    """The same layer with every gate open (Delta = -inf): the method's own claim is the ratio."""
    lb.set_density(1.0)
    d1_ms, st1 = time_layer(lb, reps, no_graph)
    lb.set_density(target)
    rec["us_density1"] = round(d1_ms * 1e3, 2)
    rec["speedup_vs_density1"] = round(d1_ms * 1e3 / rec["us"], 3)
    dense_flops = 2.0 * st1.dense_macs / max(st1.calls, 1)
    rec["dense_frac_of_tensor_peak_at_density1"] = round(
        dense_flops / (d1_ms * 1e-3) / (peaks["bf16_tflops"] * 1e12), 3)
    rec["executed_over_dense_at_density1"] = round(st1.executed_macs / max(st1.dense_macs, 1), 3)
    return rec


# Extra measurement blocks of the default run (each: every layer shape, one launch configuration
# per density; kernel times only).  The headline value stays on the workload given by --workload.
EXTRA_BLOCKS = [
    {"workload": "imagenet", "groups": 4, "rho": 0.0, "dtype": "bf16", "densities": [0.1, 0.3, 0.6, 1.0]},
    {"workload": "imagenet", "groups": 8, "rho": 0.0, "dtype": "bf16", "densities": [0.3, 1.0]},
    {"workload": "imagenet", "groups": 4, "rho": 0.5, "dtype": "bf16", "densities": [0.1, 0.3]},
    {"workload": "imagenet", "groups": 4, "rho": 0.0, "dtype": "i8", "densities": [0.3, 1.0]},
]


def run_block(block, args, peaks, rank):
    from paper_1805_12549_b200 import synth
    if block["workload"] == "imagenet":
        name = "imagenet_resnet18_gated_3x3_layers"
        shapes = synth.imagenet_resnet18_layers(64, block["groups"], transitions=block["dtype"] == "bf16")
    else:
        name = "cifar_resnet18_gated_3x3_layers"
        shapes = synth.cifar_resnet18_layers(256, block["groups"])
    out = {"workload": name, "batch": shapes[0].n, "groups": block["groups"], "rho": block["rho"],
           "dtype": block["dtype"], "densities": {}}
    per_density = {d: [] for d in block["densities"]}
    for s in shapes:
        lb = LayerBench(s, block["rho"], args.cond_mode, rank, dtype=block["dtype"])
        for d in block["densities"]:
            lb.set_density(d)
            ms, st = time_layer(lb, 3, args.no_graph)
            per_density[d].append(layer_record(lb, ms, st, peaks))
        lb.close()
        del lb
    t1 = sum(r["us"] for r in per_density[1.0]) if 1.0 in per_density else None
    for d in block["densities"]:
        recs = per_density[d]
        tot = sum(r["us"] for r in recs)
        entry = {"us_all_layers": round(tot, 2), "layers": recs}
        if t1 is not None:
            entry["speedup_vs_density1"] = round(t1 / tot, 3)
        out["densities"][str(d)] = entry
    return out


def run_network_block(args, peaks):
    """Whole CG-ResNet-18 forward pass (batch 128, 224 x 224, G = 4) at the gate density that gives a
    2.8x reduction of the network's multiplications, and the same network with every gate open."""
    import torch
    from paper_1805_12549_b200 import resnet18 as R
    batch, reduction = 128, 2.8
    net = R.CgResNet18(groups=4, cond_mode=args.cond_mode)
    gated, other = net.macs_per_image()
    tau = R.density_for_reduction(reduction, 4, gated, other)
    x = R.synthetic_images("bench_resnet18", batch)
    net.calibrate(x[:CALIB_IMAGES].contiguous(), tau)
    inst = net.instance(batch)
    stream = torch.cuda.current_stream()

    def timed(reps):
        inst.forward(x)
        torch.cuda.synchronize()
        g = capture(lambda: inst.forward(x), args.no_graph)
        g.replay()
        torch.cuda.synchronize()
        inst.stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        _, summary = inst.stats()
        return e0.elapsed_time(e1) / reps, summary

    reps = 10
    ms, summ = timed(reps)
    events = []
    for _ in range(3):
        inst.forward(x, events=events)
    torch.cuda.synchronize()
    inst.stats()
    per_op = {}
    for name, e0, e1 in events:
        per_op[name] = per_op.get(name, 0.0) + e0.elapsed_time(e1) / 3
    gated_names = {s.name for s in net.gated_specs}
    net.set_density(1.0)
    ms1, summ1 = timed(reps)
    net.set_density(tau)
    out = {
        "workload": "cg_resnet18_forward", "batch": batch, "image": 224, "groups": 4, "dtype": "bf16",
        "target_flop_reduction": reduction, "target_density": round(tau, 4),
        "calibration": f"layer by layer on the first {CALIB_IMAGES} images",
        "ms_per_forward": round(ms, 4), "images_per_s": round(batch / (ms * 1e-3), 1),
        "ms_per_forward_density1": round(ms1, 4), "images_per_s_density1": round(batch / (ms1 * 1e-3), 1),
        "speedup_vs_density1": round(ms1 / ms, 3),
        "flop_reduction": round(summ["flop_reduction"], 3),
        "gated_layer_density": round(summ["gated_layer_density"], 4),
        "executed_over_gated": round(summ["executed_macs"] / max(summ["gated_macs"], 1), 3),
        "gated_tflops": round(2.0 * summ["gated_macs"] / (ms * 1e-3) / 1e12, 1),
        "dense_tflops_density1": round(2.0 * summ1["dense_macs"] / (ms1 * 1e-3) / 1e12, 1),
        "launches_per_forward": inst.launches_per_forward(),
        "ms_gated_layers": round(sum(v for k, v in per_op.items() if k in gated_names), 4),
        "ms_other_operators": round(sum(v for k, v in per_op.items() if k not in gated_names), 4),
        "ms_per_operator": {k: round(v, 4) for k, v in per_op.items()},
        "kernels": {s.name: KERNEL_NAMES[inst.convs[s.name].kernel_id]
                    for s in net.specs},
    }
    inst.close()
    # batch-1 latency (the regime of the paper's accelerator, Table 4): the same network and
    # calibration, one image, CUDA-graph replay
    inst1 = net.instance(1)
    x1 = x[:1].contiguous()

    def latency(reps=20):
        inst1.forward(x1)
        torch.cuda.synchronize()
        g = capture(lambda: inst1.forward(x1), args.no_graph)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    out["batch1_latency_ms"] = round(latency(), 4)
    net.set_density(1.0)
    out["batch1_latency_ms_density1"] = round(latency(), 4)
    net.set_density(tau)
    inst1.close()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    wname, shapes = workload_layers(args.workload, args.batch)
    if args.layers:
        keep = set(args.layers.split(","))
        shapes = [s for s in shapes if s.name in keep]
    layers = [LayerBench(s, args.rho, args.cond_mode, rank, host=True) for s in shapes]
    for lb in layers:
        lb.set_density(args.density)
    stream = torch.cuda.current_stream()

    def step(i):
        for lb in layers:
            lb.forward(i)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(LayerBench.SETS):
        step(i)                                   # first calls encode the tensor maps
    torch.cuda.synchronize()
    step_graphs = [capture(lambda k=k: step(k), args.no_graph) for k in range(LayerBench.SETS)]

    # warm-up (at least W steps and about a second of load, so the clock samples are under load)
    sampler = ClockSampler(local) if rank == 0 else None
    t_load0 = time.time()
    for i in range(max(args.warmup, 3)):
        step_graphs[i % LayerBench.SETS].replay()
    torch.cuda.synchronize()
    while time.time() - t_load0 < 1.0:
        for i in range(40):
            step_graphs[i % LayerBench.SETS].replay()
        torch.cuda.synchronize()
    for lb in layers:
        lb.conv.stats()

    # timed region: exactly K steps, device-timed as a whole
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step_graphs[i % LayerBench.SETS].replay()
    e1.record(stream)
    torch.cuda.synchronize()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    for lb in layers:
        lb.stats = lb.conv.stats()
    ms_step = ms_total / args.steps
    batch = shapes[0].n
    value = whole_job_rate(batch, world, ms_step)

    # per-layer kernel durations at the target density and with every gate open
    reps = max(1, args.steps // LayerBench.SETS)
    per_layer = []
    for lb in layers:
        d_ms, st = time_layer(lb, reps, args.no_graph)
        rec = layer_record(lb, d_ms, st, peaks)
        per_layer.append(with_density1(lb, rec, reps, args.no_graph, peaks, args.density))
    t1 = time.time()
    clocks = sampler.stop(t_load0, t1) if sampler else None
    speedup = round(sum(r["us_density1"] for r in per_layer) / sum(r["us"] for r in per_layer), 3)
    dom = max(range(len(layers)), key=lambda j: per_layer[j]["us"])
    dl, dp = layers[dom], per_layer[dom]
    if dp["bound"] == "hbm":
        roof = {"bound": "hbm", "achieved": dp["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": dp["gated_tflops"], "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s"}
    roof["frac"] = round(roof["achieved"] / roof["peak"], 4)
    roof["traffic"] = measured_traffic(dp["layer"])
    roof["algorithmic_bytes"] = dl.algorithmic_bytes
    roof["kernel"] = f"{dp['kernel']} ({dp['layer']})"
    roof["peak_source"] = f"of {peaks['source']}"
    roof["us_per_launch"] = dp["us"]

    # end to end: host buffers through the C ABI, copies inside the timed region.  The layers of a
    # step are independent, so each runs on its own stream: the host-to-device copy of one layer
    # overlaps the device-to-host copy of another (PCIe is full duplex); e0 and e1 bracket all of them.
    e2e_steps = max(3, min(args.steps, 20))
    side = [torch.cuda.Stream() for _ in layers]
    for lb in layers:
        lb.forward_host()
    barrier()
    e0.record(stream)
    for st in side:
        st.wait_event(e0)
    for _ in range(e2e_steps):
        for lb, st in zip(layers, side):
            lb.forward_host(st)
    for st in side:
        done = torch.cuda.Event()
        done.record(st)
        stream.wait_event(done)
    e1.record(stream)
    torch.cuda.synchronize()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1))
    for lb in layers:
        lb.conv.stats()
    e2e = {"value": round(whole_job_rate(batch, world, ms_e2e / e2e_steps), 1), "unit": UNIT,
           "h2d_bytes_per_step": sum(lb.bytes_x for lb in layers),
           "d2h_bytes_per_step": sum(lb.bytes_y + lb.bytes_mask for lb in layers)}
    launches = args.steps * sum(lb.B.cg_conv_launches_per_forward(lb.conv.handle) for lb in layers)
    for lb in layers:
        lb.close()
    del layers, step_graphs
    torch.cuda.empty_cache()

    blocks = []
    if rank == 0 and world == 1 and not args.no_extra:
        for block in EXTRA_BLOCKS:
            blocks.append(run_block(block, args, peaks, rank))
            torch.cuda.empty_cache()
        blocks.append(run_network_block(args, peaks))
        torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(args, shapes)

    if rank == 0:
        out = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 5),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": wname, "batch_per_gpu": batch, "groups": 4,
                       "target_density": args.density, "rho": args.rho,
                       "cond_mode": args.cond_mode,
                       "calibration": f"gate statistics and Delta from the first {CALIB_IMAGES} images",
                       "l2": f"x/y/mask rotate over {LayerBench.SETS} buffer sets per layer "
                             "(total > L2)", "parallelism": f"batch x{world}, no collective",
                       "e2e": "host buffers through cg_conv_forward_host, one stream per layer"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "speedup_vs_density1": speedup,
            "roofline": roof, "cpu_baseline": cpu, "layers": per_layer, "blocks": blocks,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------- oracle arm
def oracle_layer_inputs(s, density, rho, images):
    """The same seeded layer as LayerBench, cut to `images` images; gate statistics and Delta from
    the oracle's partial sums of the first CALIB_IMAGES images (the direct kernels that calibrate
    the other arm reproduce these sums bit for bit)."""
    from oracle import oracle as O
    from paper_1805_12549_b200 import synth
    key = ("bench", s.name, 0)
    chunk = 16
    n_need = max(images, min(CALIB_IMAGES, s.n))
    n_gen = ((n_need + chunk - 1) // chunk) * chunk
    x_all = synth.bf16_round(synth.smoothed_noise((key, "x"), min(n_gen, s.n), s.hw, s.hw, s.c_in,
                                                  rho=rho))
    wb, wc = synth.kaiming_weights(key, s.c_out, 3, 3, s.c_in, s.groups)
    wb, wc = synth.bf16_round(wb), synth.bf16_round(wc)
    bn = synth.bn_params(key, s.c_out)
    calib = min(CALIB_IMAGES, s.n)
    sh = O.Shape(images, s.hw, s.hw, s.c_in, s.c_out, stride=s.stride, groups=s.groups)
    cs = O.Shape(calib, s.hw, s.hw, s.c_in, s.c_out, stride=s.stride, groups=s.groups)
    probe = O.gated_conv(cs, x_all[:calib], wb, wc, bn, np.full(s.c_out, np.inf, np.float32))
    bn["gate_mean"], bn["gate_var"], p_hat = calibrate(probe.p.reshape(-1, s.c_out), None)
    dval = delta_for(p_hat, density)
    return sh, x_all[:images], wb, wc, bn, np.full(s.c_out, dval, np.float32)


def cpu_baseline(args, shapes):
    """The oracle, as it stands, on the host cores: the first `images` images of the batch
    through every layer shape, repeated for about ten seconds; the best pass is reported."""
    from oracle import oracle as O
    images = args.cpu_images or shapes[0].n
    prepared = [oracle_layer_inputs(s, args.density, args.rho, images) for s in shapes]
    times, t_all = [], time.time()
    while len(times) < 8 and (not times or time.time() - t_all < 10.0):
        t0 = time.time()
        for sh, x, wb, wc, bn, delta in prepared:
            O.gated_conv(sh, x, wb, wc, bn, delta, out_bf16=True)
        times.append(time.time() - t0)
    dt = min(times)
    return {"value": round(images / dt, 3), "unit": UNIT, "cores": O.num_threads(),
            "kind": "oracle",
            "sample": f"first {images} images of the batch through every layer shape, best of "
                      f"{len(times)} passes ({sum(times):.1f} s of CPU work)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    wname, shapes = workload_layers(args.workload, args.batch)
    from oracle import oracle as O
    images = args.cpu_images or shapes[0].n
    prepared = [oracle_layer_inputs(s, args.density, args.rho, images) for s in shapes]

    def step():
        for sh, x, wb, wc, bn, delta in prepared:
            O.gated_conv(sh, x, wb, wc, bn, delta, out_bf16=True)

    # keep the whole run within a few minutes: cap steps by a time budget
    t_probe = time.time()
    step()
    per = time.time() - t_probe
    warm = max(0, min(args.warmup, int(20.0 / max(per, 1e-3))) - 1)
    steps = max(1, min(args.steps, int(120.0 / max(per, 1e-3))))
    for _ in range(warm):
        step()
    t0 = time.time()
    for _ in range(steps):
        step()
    dt = (time.time() - t0) / steps
    value = images / dt
    sample = f"each step = first {images} images of the batch through every layer shape"
    out = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT,
           "n_gpus": args.gpus, "steps": steps, "warmup": warm + 1,
           "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": wname, "batch_per_gpu": shapes[0].n, "groups": 4,
                      "target_density": args.density, "rho": args.rho, "sample": sample},
           "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": O.num_threads(),
                            "kind": "oracle", "sample": sample},
           "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0,
                   "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cifar", choices=["cifar", "imagenet"])
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--density", type=float, default=0.3)
    ap.add_argument("--rho", type=float, default=0.0)
    ap.add_argument("--cond-mode", type=int, default=0)
    ap.add_argument("--cpu-images", type=int, default=None)
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the extra blocks (ImageNet shapes, G = 8, density sweep, int8)")
    ap.add_argument("--layers", default=None,
                    help="comma-separated layer names to keep (e.g. c64@56,c256@14)")
    ap.add_argument("--no-graph", action="store_true",
                    help="plain launches instead of CUDA graphs (for profilers)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly with --gpus N: run N ranks, one per GPU (each shards nothing and
        # exchanges nothing on the data path; only the timing is reduced over the ranks)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
               f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port",
               str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    run_ours(args)


if __name__ == "__main__":
    main()
