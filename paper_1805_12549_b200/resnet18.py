"""CG-ResNet-18: a whole network of channel-gated layers driven through the C ABI.

"Channel Gating Neural Networks" (Section 5) evaluates gating on standard networks; this module
lays out a ResNet-18 for 224x224 images in which every 3x3 convolution after the stem is a
channel-gated layer (Section 3.1) with G groups, and runs its inference forward pass on the
device: every convolution is a cg_conv_forward call (include/cgconv.h), everything in between is
one of the four operators of include/cgnet.h.  Python only owns the buffers and the order of the
calls.

Layers that are not gated (the 7x7 stem, the 1x1 shortcut convolutions, the classifier) run as
layers with G = 1, where the base path is the whole convolution (Section 3.1 allows eta = 1).
The stem is computed as a patch matrix (cg_im2col_bf16) followed by a 1x1 layer over it.

Weights are random (Kaiming-normal); the batch-norm statistics, the gate statistics of Eq. 3 and
the thresholds Delta come from a layer-by-layer calibration pass over a few images, which stands
in for training: BN1 and the gate use the statistics of the partial sums P, BN2 those of the full
sums P + R (Section 4), and each gated layer's Delta is the quantile of its normalised partial
sums that gives the requested gate density.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import binding as B
from . import synth

STAGES = ((64, 1), (128, 2), (256, 2), (512, 2))   # channels, stride of the stage's first block
STEM_K, STEM_STRIDE, STEM_PAD, STEM_KPAD = 7, 2, 3, 192   # 7*7*3 = 147 patch columns, padded to 3 x 64


def density_for_reduction(reduction, groups, gated_macs, other_macs):
    """Gate density tau at which the whole network does 1/reduction of its dense multiplications:
    other + gated * (1/G + (1 - 1/G) * tau) = (other + gated) / reduction  (FLOP model of
    Section 3.1: the base path always runs, the conditional path where the gate fires)."""
    eta = 1.0 / groups
    frac = ((other_macs + gated_macs) / reduction - other_macs) / gated_macs
    return float(min(max((frac - eta) / (1.0 - eta), 0.0), 1.0))


@dataclass
class ConvSpec:
    name: str
    c_in: int
    c_out: int
    k: int
    stride: int
    pad: int
    groups: int
    relu: bool
    has_residual: bool
    h: int                      # input extent (square)
    true_macs_per_image: int    # multiplications of the convolution this layer stands for
    gated: bool = False
    # parameters (device tensors), filled by CgResNet18
    wb: torch.Tensor = None
    wc: torch.Tensor = None
    params: dict = field(default_factory=dict)
    delta: torch.Tensor = None
    bn: B.CgBnParams = None
    p_hat: np.ndarray = None    # normalised partial sums of the calibration images

    @property
    def ho(self):
        return (self.h + 2 * self.pad - self.k) // self.stride + 1


def _dev_bf16(a):
    bits = synth.bf16_bits(np.ascontiguousarray(a, np.float32)).view(np.int16)
    return torch.from_numpy(bits).cuda().view(torch.bfloat16)


class CgResNet18:
    def __init__(self, image=224, groups=4, classes=1000, key=("cg_resnet18",), cond_mode=B.CG_COND_AUTO,
                 algo=B.CG_ALGO_AUTO):
        self.image, self.groups, self.classes, self.key = image, groups, classes, key
        self.cond_mode, self.algo = cond_mode, algo
        self.specs = []
        h = (image + 2 * STEM_PAD - STEM_K) // STEM_STRIDE + 1
        self.stem_hw = h
        self._add("stem", STEM_KPAD, 64, 1, 1, 0, 1, True, False, h, STEM_K * STEM_K * 3 * 64 * h * h)
        h = (h + 2 - 3) // 2 + 1                      # max pooling 3x3, stride 2, padding 1
        c = 64
        self.blocks = []                              # (shortcut spec or None, conv1, conv2)
        for si, (co, stride) in enumerate(STAGES):
            for bi in range(2):
                st = stride if bi == 0 else 1
                ho = (h + 2 - 3) // st + 1
                short = None
                if st != 1 or c != co:
                    short = self._add(f"layer{si + 1}.{bi}.shortcut", c, co, 1, 1, 0, 1, False, False, ho,
                                      c * co * ho * ho)
                c1 = self._add(f"layer{si + 1}.{bi}.conv1", c, co, 3, st, 1, groups, True, False, h,
                               9 * c * co * ho * ho, gated=True)
                c2 = self._add(f"layer{si + 1}.{bi}.conv2", co, co, 3, 1, 1, groups, True, True, ho,
                               9 * co * co * ho * ho, gated=True)
                self.blocks.append((short, c1, c2, st))
                c, h = co, ho
        self.final_hw = h
        # the classifier's columns are padded with zero filters to a multiple of 64 (tensor-core kernels)
        self.fc = self._add("fc", c, (classes + 63) // 64 * 64, 1, 1, 0, 1, False, False, 1, c * classes)
        self._init_params()

    # ------------------------------------------------------------------ construction
    def _add(self, name, c_in, c_out, k, stride, pad, groups, relu, has_res, h, macs, gated=False):
        s = ConvSpec(name, c_in, c_out, k, stride, pad, groups, relu, has_res, h, macs, gated)
        self.specs.append(s)
        return s

    def _init_params(self):
        for s in self.specs:
            key = (*self.key, s.name)
            if s.name == "stem":
                # the 7x7x3 filter, flattened in (r, s, c) order and zero-padded to the patch width
                w, _ = synth.kaiming_weights(key, s.c_out, STEM_K, STEM_K, 3, 1)
                wp = np.zeros((s.c_out, 1, 1, STEM_KPAD), np.float32)
                wp[:, 0, 0, :STEM_K * STEM_K * 3] = w.reshape(s.c_out, -1)
                self.stem_filter = w
                wb, wc = wp, np.zeros((s.c_out, 1, 1, 0), np.float32)
            else:
                wb, wc = synth.kaiming_weights(key, s.c_out, s.k, s.k, s.c_in, s.groups)
            if s.name == "fc":
                wb[self.classes:] = 0.0
            s.wb = _dev_bf16(wb)
            s.wc = _dev_bf16(wc) if wc.size else None
            bn = synth.bn_params(key, s.c_out)
            one, zero = np.ones(s.c_out, np.float32), np.zeros(s.c_out, np.float32)
            if s.name == "fc":                        # plain affine classifier: y = W x + bias
                bn["gamma"], bn["beta"] = one, bn["beta"]
            names = ("gamma", "beta", "mean_base", "var_base", "mean_full", "var_full", "gate_mean", "gate_var")
            vals = dict(gamma=bn["gamma"], beta=bn["beta"], mean_base=zero, var_base=one, mean_full=zero,
                        var_full=one, gate_mean=zero, gate_var=one)
            s.params = {k: torch.from_numpy(vals[k].copy()).cuda() for k in names}
            s.bn = B.make_bn(s.params)
            # ungated layers: the gate never fires, y = f(BN1(P)) with P the whole convolution
            s.delta = torch.full((s.c_out,), float("inf") if not s.gated else 0.0, dtype=torch.float32,
                                 device="cuda")

    @property
    def gated_specs(self):
        return [s for s in self.specs if s.gated]

    def macs_per_image(self):
        gated = sum(s.true_macs_per_image for s in self.specs if s.gated)
        other = sum(s.true_macs_per_image for s in self.specs if not s.gated)
        return gated, other

    def instance(self, n):
        return Instance(self, n)

    # ------------------------------------------------------------------ calibration
    def calibrate(self, x_cal, density):
        """Layer by layer over the images x_cal [n,image,image,3] (bf16, device): sets every
        layer's batch-norm and gate statistics from its own sums, sets each gated layer's Delta
        for `density`, then runs the layer to get the next layer's input."""
        inst = Instance(self, x_cal.shape[0])
        inst.forward(x_cal, before_conv=self._calibrate_layer, density=density)
        torch.cuda.synchronize()
        inst.close()

    def _calibrate_layer(self, s: ConvSpec, x, n, density):
        eps = 1e-5
        cal = B.GatedConv(n, s.h, s.h, s.c_in, s.c_out, k=s.k, stride=s.stride, pad=s.pad, groups=s.groups,
                          dtype=B.CG_BF16, algo=B.CG_ALGO_DIRECT)
        p = torch.empty((cal.m, s.c_out), dtype=torch.float32, device="cuda")
        B.cg_conv_partial_sums(cal.handle, x, s.wb, p)
        torch.cuda.synchronize()
        cal.close()
        pn = p.cpu().numpy().astype(np.float64)
        mean = pn.mean(0).astype(np.float32)
        var = np.maximum(pn.var(0), 1e-6).astype(np.float32)
        if s.name == "fc":                            # no normalisation in front of the classifier
            mean, var = np.zeros_like(mean), np.ones_like(var)
        for k, v in (("mean_base", mean), ("var_base", var), ("gate_mean", mean), ("gate_var", var),
                     ("mean_full", mean), ("var_full", var)):
            s.params[k].copy_(torch.from_numpy(v))
        if not s.gated:
            return
        s.p_hat = ((pn - mean) / np.sqrt(var.astype(np.float64) + eps)).ravel()
        # statistics of the full sums P + R: the layer with every gate open, no batch norm, no ReLU
        full = B.GatedConv(n, s.h, s.h, s.c_in, s.c_out, k=s.k, stride=s.stride, pad=s.pad, groups=s.groups,
                           dtype=B.CG_BF16, relu=False, bn_eps=0.0, algo=self.algo, cond_mode=B.CG_COND_DENSE)
        one = torch.ones(s.c_out, device="cuda")
        zero = torch.zeros(s.c_out, device="cuda")
        ident = dict(gamma=one, beta=zero, mean_base=zero, var_base=one, mean_full=zero, var_full=one)
        y, _ = full.alloc_outputs()
        full.forward(x, s.wb, s.wc, B.make_bn(ident), torch.full((s.c_out,), float("-inf"), device="cuda"), y)
        torch.cuda.synchronize()
        full.close()
        yn = y.float().reshape(-1, s.c_out).cpu().numpy().astype(np.float64)
        s.params["mean_full"].copy_(torch.from_numpy(yn.mean(0).astype(np.float32)))
        s.params["var_full"].copy_(torch.from_numpy(np.maximum(yn.var(0), 1e-6).astype(np.float32)))
        self.set_density(density, [s])

    def set_density(self, density, specs=None):
        """Rewrites Delta of the gated layers in place (captured graphs read the new values)."""
        for s in specs or self.gated_specs:
            if density >= 1.0:
                d = float("-inf")
            elif density <= 0.0:
                d = float("inf")
            else:
                d = float(np.quantile(s.p_hat, 1.0 - density))
            s.delta.fill_(d)


class Instance:
    """Handles and activation buffers of the network for one batch size."""

    def __init__(self, net: CgResNet18, n: int):
        self.net, self.n = net, n
        bf = dict(dtype=torch.bfloat16, device="cuda")
        self.patches = torch.empty((n, net.stem_hw, net.stem_hw, STEM_KPAD), **bf)
        self.convs, self.out, self.mask = {}, {}, {}
        for s in net.specs:
            algo = net.algo
            if s.c_out % 32 or s.c_in % 64:
                algo = B.CG_ALGO_AUTO
            conv = B.GatedConv(n, s.h, s.h, s.c_in, s.c_out, k=s.k, stride=s.stride, pad=s.pad,
                               groups=s.groups, dtype=B.CG_BF16, relu=s.relu, has_residual=s.has_residual,
                               algo=algo, cond_mode=net.cond_mode)
            self.convs[s.name] = conv
            y, mask = conv.alloc_outputs()
            self.out[s.name] = y
            self.mask[s.name] = mask if s.gated else None
        hp = (net.stem_hw + 2 - 3) // 2 + 1
        self.pooled = torch.empty((n, hp, hp, 64), **bf)
        self.sub = {sh.name: torch.empty((n, sh.h, sh.h, sh.c_in), **bf) for sh, _, _, _ in net.blocks if sh}
        self.avg = torch.empty((n, 1, 1, net.fc.c_in), **bf)
        self.launches = None

    def _conv(self, s, x, residual, before_conv, density, record):
        if before_conv is not None:
            before_conv(s, x, self.n, density)
        y = self.out[s.name]
        self.convs[s.name].forward(x, s.wb, s.wc, s.bn, s.delta, y, self.mask[s.name], residual)
        if record is not None:
            record.append((s, x.clone(), None if residual is None else residual.clone(), y.clone(),
                           None if self.mask[s.name] is None else self.mask[s.name].clone()))
        return y

    def forward(self, x, before_conv=None, density=None, record=None, events=None):
        """x [n,image,image,3] bf16 -> logits [n,classes] bf16 (a view of an owned buffer).
        `events`, a list, receives (operator name, start event, end event) per call."""
        net = self.net

        def timed(name, fn):
            if events is None:
                return fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            out = fn()
            e1.record()
            events.append((name, e0, e1))
            return out

        go = lambda s, a, r=None: timed(s.name, lambda: self._conv(s, a, r, before_conv, density, record))
        timed("stem.im2col", lambda: B.cg_im2col_bf16(x, self.patches, STEM_K, STEM_STRIDE, STEM_PAD))
        a = go(net.specs[0], self.patches)
        timed("maxpool", lambda: B.cg_maxpool_bf16(a, self.pooled, 3, 2, 1))
        a = self.pooled
        for short, c1, c2, st in net.blocks:
            identity = a
            if short is not None:
                src = a
                if st != 1:
                    timed(short.name + ".subsample", lambda: B.cg_subsample_bf16(a, self.sub[short.name], st))
                    src = self.sub[short.name]
                identity = go(short, src)
            t = go(c1, a)
            a = go(c2, t, identity)
        timed("avgpool", lambda: B.cg_avgpool_bf16(a, self.avg))
        logits = go(net.fc, self.avg)
        return logits.view(self.n, net.fc.c_out)[:, :net.classes]

    def launches_per_forward(self):
        """Kernels one forward pass launches: those of every layer plus the glue operators."""
        n = sum(B.cg_conv_launches_per_forward(c.handle) for c in self.convs.values())
        return n + 3 + sum(1 for sh, _, _, st in self.net.blocks if sh is not None and st != 1)

    def stats(self):
        """Per-layer counters since the last call, and the network's FLOP summary (multiplications
        of the convolutions the layers stand for)."""
        per = {name: c.stats() for name, c in self.convs.items()}
        gated_dense = gated_done = gated_exec = other = 0
        for s in self.net.specs:
            st = per[s.name]
            calls = max(st.calls, 1)
            if s.gated:
                gated_dense += st.dense_macs // calls
                gated_done += st.gated_macs // calls
                gated_exec += st.executed_macs // calls
            else:
                other += s.true_macs_per_image * self.n
        dense = gated_dense + other
        return per, dict(dense_macs=dense, gated_macs=gated_done + other, executed_macs=gated_exec + other,
                         other_macs=other, flop_reduction=dense / max(gated_done + other, 1),
                         gated_layer_density=sum(per[s.name].active for s in self.net.gated_specs) /
                         max(sum(per[s.name].outputs for s in self.net.gated_specs), 1))

    def close(self):
        for c in self.convs.values():
            c.close()
        self.convs = {}


def synthetic_images(key, n, image=224):
    """Smoothed Gaussian noise images [n,image,image,3] as bf16 on the device (no ReLU: pixel
    values of both signs, like normalised images)."""
    x = synth.smoothed_noise((key, "images"), n, image, image, 3, relu=False)
    return _dev_bf16(x)
