#!/usr/bin/env python
"""Throughput of the channel-gated convolution layers on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload cifar|imagenet] [--density D] [--rho R] [--cond-mode M]

One step = one forward pass of every gated 3x3 layer shape of the workload over one batch
of synthetic activations (ReLU of box-smoothed Gaussian noise, bf16).  Prints ONE JSON line.
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


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the layer kernel,
# from the ncu captures summarised under profiles/.  It is reported only while the kernel sources
# still hash to what they were when the counters were taken.
TRAFFIC = {
    "source_sha": "0e2953bc28412162",
    # profiles/tc_gated_conv_kernel_c64at32_full.txt and ..._c128at16_full.txt; the y and mask writes
    # of the captured launch were still in the 126 MB L2 when it ended, so they are not in these sums
    "bytes_per_launch": {"c64@32": 33736192 + 633088, "c128@16": 17210624 + 256},
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
class LayerBench:
    """Device buffers, calibrated gate parameters and the handle of one layer shape."""

    SETS = 4   # x/y/mask buffer sets rotated so that no step finds its tensors in L2

    def __init__(self, shape, density, rho, cond_mode, rank):
        import torch
        from paper_1805_12549_b200 import binding as B, synth
        self.B, self.torch, self.shape = B, torch, shape
        s = shape
        key = ("bench", s.name, rank)
        x = synth.bf16_bits(synth.smoothed_noise((key, "x"), s.n, s.hw, s.hw, s.c_in, rho=rho))
        wb, wc = synth.kaiming_weights(key, s.c_out, 3, 3, s.c_in, s.groups)
        bn = synth.bn_params(key, s.c_out)
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
        bf = lambda a: dev(synth.bf16_bits(a).view(np.int16)).view(torch.bfloat16)
        x0 = dev(x.view(np.int16)).view(torch.bfloat16)
        self.x_host = x0.cpu().pin_memory()
        self.xs = [x0] + [torch.roll(x0, k, dims=0).contiguous() for k in range(1, self.SETS)]
        self.wb, self.wc = bf(wb), bf(wc)
        self.conv = B.GatedConv(s.n, s.hw, s.hw, s.c_in, s.c_out, k=3, stride=s.stride, pad=1,
                                groups=s.groups, dtype=B.CG_BF16, cond_mode=cond_mode)
        self.params = {k: dev(v) for k, v in bn.items()}
        # gate statistics = per-channel mean/variance of the partial sums over this batch
        # (what a trained network's running statistics would hold); Delta = one scalar per
        # layer at the quantile of the normalised partial sums that gives the target density
        p = torch.empty((self.conv.m, s.c_out), dtype=torch.float32, device="cuda")
        B.cg_conv_partial_sums(self.conv.handle, x0, self.wb, p)
        torch.cuda.synchronize()
        mean, var = p.mean(dim=0), p.var(dim=0, unbiased=False).clamp_min(1e-6)
        self.params["gate_mean"], self.params["gate_var"] = mean.contiguous(), var.contiguous()
        if density >= 1.0:
            dval = float("-inf")
        else:
            p_hat = ((p - mean) / torch.sqrt(var + 1e-5)).flatten()
            idx = torch.randint(0, p_hat.numel(), (min(p_hat.numel(), 4_000_000),), device="cuda")
            dval = float(torch.quantile(p_hat[idx], 1.0 - density))
        del p
        self.delta = torch.full((s.c_out,), dval, dtype=torch.float32, device="cuda")
        self.bn = B.make_bn(self.params)
        self.ys, self.masks = zip(*[self.conv.alloc_outputs() for _ in range(self.SETS)])
        self.y_host = torch.empty(self.ys[0].shape, dtype=torch.bfloat16).pin_memory()
        self.mask_host = torch.empty(self.masks[0].shape, dtype=torch.int32).pin_memory()
        self.staging = torch.empty(B.cg_conv_host_staging_bytes(self.conv.handle),
                                   dtype=torch.uint8, device="cuda")
        el = 2
        self.bytes_x = s.n * s.hw * s.hw * s.c_in * el
        self.bytes_y = self.conv.m * s.c_out * el
        self.bytes_mask = self.conv.m * self.conv.words * 4
        self.bytes_w = s.c_out * 9 * s.c_in * el
        self.algorithmic_bytes = self.bytes_x + self.bytes_y + self.bytes_mask + self.bytes_w
        self.stats = None

    def forward(self, i):
        k = i % self.SETS
        self.conv.forward(self.xs[k], self.wb, self.wc, self.bn, self.delta, self.ys[k],
                          self.masks[k])

    def forward_host(self):
        self.B.cg_conv_forward_host(self.conv.handle, self.x_host, self.wb, self.wc, self.bn,
                                    self.delta, None, self.y_host, self.mask_host, self.staging)


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
    layers = [LayerBench(s, args.density, args.rho, args.cond_mode, rank) for s in shapes]
    stream = torch.cuda.current_stream()

    def step(i):
        for lb in layers:
            lb.forward(i)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # Launches go through CUDA graphs (one graph = one step on one buffer set), so the
    # device, not the Python caller, sets the pace.
    class Plain:
        def __init__(self, fn):
            self.fn = fn

        def replay(self):
            self.fn()

    def capture(fn):
        if args.no_graph:
            return Plain(fn)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    for i in range(LayerBench.SETS):
        step(i)                                   # first calls encode the tensor maps
    torch.cuda.synchronize()
    step_graphs = [capture(lambda k=k: step(k)) for k in range(LayerBench.SETS)]
    layer_graphs = [capture(lambda lb=lb: [lb.forward(k) for k in range(LayerBench.SETS)])
                    for lb in layers]

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
    t1 = time.time()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    for lb in layers:
        lb.stats = lb.conv.stats()
    ms_step = ms_total / args.steps
    batch = shapes[0].n
    value = whole_job_rate(batch, world, ms_step)

    # per-layer kernel durations: the same launches, one layer at a time, back to back
    reps = max(1, args.steps // LayerBench.SETS)
    layer_ms = []
    for g in layer_graphs:
        g.replay()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        layer_ms.append(e0.elapsed_time(e1) / (reps * LayerBench.SETS))
    t1 = time.time()
    clocks = sampler.stop(t_load0, t1) if sampler else None
    for lb in layers:
        lb.conv.stats()

    per_layer = []
    for j, lb in enumerate(layers):
        d_ms = layer_ms[j]
        st = lb.stats
        dens = st.density
        flops = 2.0 * st.gated_macs / max(st.calls, 1)
        t_tensor = flops / (peaks["bf16_tflops"] * 1e12)
        t_hbm = lb.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9)
        per_layer.append({
            "layer": lb.shape.name, "us": round(d_ms * 1e3, 2), "density": round(dens, 4),
            "tensor_cores": bool(lb.conv.uses_tensor_cores),
            "gated_tflops": round(flops / (d_ms * 1e-3) / 1e12, 1),
            "gbs": round(lb.algorithmic_bytes / (d_ms * 1e-3) / 1e9, 1),
            "roof_us": round(max(t_tensor, t_hbm) * 1e6, 2),
            "roof_frac": round(max(t_tensor, t_hbm) / (d_ms * 1e-3), 3),
            "bound": "tensor" if t_tensor > t_hbm else "hbm",
            "flop_reduction": round(st.dense_macs / max(st.gated_macs, 1), 3),
            "executed_over_gated": round(st.executed_macs / max(st.gated_macs, 1), 3),
            "blocks_skipped": f"{st.tiles_skipped}/{st.tiles_total}",
        })
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
    roof["kernel"] = f"tc_gated_conv_kernel ({dp['layer']})"
    roof["peak_source"] = f"of {peaks['source']}"
    roof["us_per_launch"] = dp["us"]

    # end to end: host buffers through the C ABI, copies inside the timed region
    e2e_steps = max(3, min(args.steps, 20))
    for lb in layers:
        lb.forward_host()
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        for lb in layers:
            lb.forward_host()
    e1.record(stream)
    torch.cuda.synchronize()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1))
    for lb in layers:
        lb.conv.stats()
    e2e = {"value": round(whole_job_rate(batch, world, ms_e2e / e2e_steps), 1), "unit": UNIT,
           "h2d_bytes_per_step": sum(lb.bytes_x for lb in layers),
           "d2h_bytes_per_step": sum(lb.bytes_y + lb.bytes_mask for lb in layers)}

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
                       "l2": f"x/y/mask rotate over {LayerBench.SETS} buffer sets per layer "
                             "(total > L2)", "parallelism": f"batch x{world}, no collective"},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": args.steps * sum(lb.B.cg_conv_launches_per_forward(lb.conv.handle)
                                             for lb in layers),
            "roofline": roof, "cpu_baseline": cpu, "layers": per_layer,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------- oracle arm
def oracle_layer_inputs(s, density, rho, images):
    """The same seeded layer as LayerBench, cut to `images` images, calibrated by the oracle."""
    from oracle import oracle as O
    from paper_1805_12549_b200 import synth
    key = ("bench", s.name, 0)
    chunk = 16
    n_gen = ((images + chunk - 1) // chunk) * chunk
    x = synth.bf16_round(synth.smoothed_noise((key, "x"), min(n_gen, s.n), s.hw, s.hw, s.c_in,
                                              rho=rho))[:images]
    wb, wc = synth.kaiming_weights(key, s.c_out, 3, 3, s.c_in, s.groups)
    wb, wc = synth.bf16_round(wb), synth.bf16_round(wc)
    bn = synth.bn_params(key, s.c_out)
    sh = O.Shape(images, s.hw, s.hw, s.c_in, s.c_out, stride=s.stride, groups=s.groups)
    one = O.Shape(1, s.hw, s.hw, s.c_in, s.c_out, stride=s.stride, groups=s.groups)
    probe = O.gated_conv(one, x[:1], wb, wc, bn, np.full(s.c_out, np.inf, np.float32))
    p = probe.p.reshape(-1, s.c_out).astype(np.float64)
    bn["gate_mean"] = p.mean(0).astype(np.float32)
    bn["gate_var"] = np.maximum(p.var(0), 1e-6).astype(np.float32)
    if density >= 1.0:
        dval = -np.inf
    else:
        p_hat = (p - bn["gate_mean"]) / np.sqrt(bn["gate_var"] + 1e-5)
        dval = float(np.quantile(p_hat, 1.0 - density))
    return sh, x, wb, wc, bn, np.full(s.c_out, dval, np.float32)


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
    ap.add_argument("--layers", default=None,
                    help="comma-separated layer names to keep (e.g. c64@56,c256@14)")
    ap.add_argument("--no-graph", action="store_true",
                    help="plain launches instead of CUDA graphs (for profilers)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
