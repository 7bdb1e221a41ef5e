"""Seeded synthetic inputs for the channel-gated convolution layer.

This module only DRAWS DATA.  It holds none of the layer's arithmetic (no
convolution, no gate, no batch norm): the CUDA library and the CPU oracle are
both fed from here and share nothing else.

The workloads stand in for the activations of CIFAR-10 / ImageNet ResNet-18
layers (the paper's Section 5 models), whose data sets and trained weights are
not available: only the layer shapes are kept.  Activations are the ReLU of
Gaussian noise smoothed by a 5x5 box filter, so that gate masks come out
spatially clustered, as the paper's computation-intensity maps (Fig. 2) show
for trained networks.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass

import numpy as np

BASE_SEED = 180512549


def rng(*key) -> np.random.Generator:
    """Counter-based generator keyed by (config, layer, tensor name, ...)."""
    h = zlib.crc32(repr(key).encode())
    return np.random.Generator(np.random.Philox(key=[BASE_SEED, h]))


# --------------------------------------------------------------------------- dtype helpers
def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bfloat16, kept as float32."""
    return bf16_to_f32(bf16_bits(a))


# --------------------------------------------------------------------------- activations
def _box5(a: np.ndarray) -> np.ndarray:
    """5x5 box mean over (H, W) of an [N,H,W,C] array with zero padding."""
    n, h, w, c = a.shape
    p = np.zeros((n, h + 4, w + 4, c), a.dtype)
    p[:, 2:-2, 2:-2, :] = a
    rows = p[:, 0:h] + p[:, 1:h + 1] + p[:, 2:h + 2] + p[:, 3:h + 3] + p[:, 4:h + 4]
    out = rows[:, :, 0:w] + rows[:, :, 1:w + 1] + rows[:, :, 2:w + 2] + rows[:, :, 3:w + 3] \
        + rows[:, :, 4:w + 4]
    return out / np.float32(25.0)


def smoothed_noise(key, n, h, w, c, rho=0.0, relu=True, chunk=16) -> np.ndarray:
    """ReLU(5 * box5(g)), g ~ N(0,1) per (n,h,w,c).

    rho in [0,1] mixes in a noise field shared by all channels of a pixel:
    g = sqrt(rho)*g_shared[n,h,w] + sqrt(1-rho)*g_own[n,h,w,c].  rho = 0 is the
    plain reading of "Gaussian noise smoothed by a 5x5 box filter"; rho > 0 makes
    the gates of different output channels fire together at a pixel.
    The factor 5 restores roughly unit variance after the 25-tap mean.
    """
    out = np.empty((n, h, w, c), np.float32)
    for i0 in range(0, n, chunk):
        i1 = min(n, i0 + chunk)
        g = rng(key, "own", i0).standard_normal((i1 - i0, h, w, c), dtype=np.float32)
        if rho > 0.0:
            sh = rng(key, "shared", i0).standard_normal((i1 - i0, h, w, 1), dtype=np.float32)
            g = np.float32(np.sqrt(rho)) * sh + np.float32(np.sqrt(1.0 - rho)) * g
        v = np.float32(5.0) * _box5(g)
        if relu:
            v = np.maximum(v, np.float32(0.0))
        out[i0:i1] = v
    return out


# --------------------------------------------------------------------------- parameters
def kaiming_weights(key, c_out, kh, kw, c_in, groups):
    """W ~ N(0, 2/(kh*kw*c_in)) as [c_out,kh,kw,c_in], split along c_in into
    W_base [c_out,kh,kw,c_in/G] and W_cond [c_out,kh,kw,c_in - c_in/G]."""
    std = np.sqrt(2.0 / (kh * kw * c_in))
    w = (rng(key, "w").standard_normal((c_out, kh, kw, c_in), dtype=np.float32)
         * np.float32(std))
    cp = c_in // groups
    return np.ascontiguousarray(w[..., :cp]), np.ascontiguousarray(w[..., cp:])


def bn_params(key, c_out, separate=True) -> dict:
    """gamma ~ U(0.5,1.5), beta ~ N(0,0.1^2), running mean ~ N(0,0.1^2), running var ~
    U(0.5,1.5).  separate=False gives the base, full and gate statistics one shared draw."""
    g = rng(key, "bn")
    out = {
        "gamma": g.uniform(0.5, 1.5, c_out).astype(np.float32),
        "beta": (0.1 * g.standard_normal(c_out)).astype(np.float32),
    }
    names = ("base", "full", "gate")
    first = None
    for nm in names:
        mean = (0.1 * g.standard_normal(c_out)).astype(np.float32)
        var = g.uniform(0.5, 1.5, c_out).astype(np.float32)
        if not separate:
            if first is None:
                first = (mean, var)
            mean, var = first
        if nm == "gate":
            out["gate_mean"], out["gate_var"] = mean, var
        else:
            out["mean_" + nm], out["var_" + nm] = mean, var
    return out


def residual(key, shape) -> np.ndarray:
    return rng(key, "res").standard_normal(shape, dtype=np.float32)


# --------------------------------------------------------------------------- int8 workload
def int8_activations(key, n, h, w, c) -> np.ndarray:
    return rng(key, "x8").integers(0, 128, (n, h, w, c), dtype=np.int8)


def int8_weights(key, c_out, kh, kw, c_in, groups):
    w = rng(key, "w8").integers(-127, 128, (c_out, kh, kw, c_in), dtype=np.int8)
    cp = c_in // groups
    return np.ascontiguousarray(w[..., :cp]), np.ascontiguousarray(w[..., cp:])


def int8_requant(key, c_out, shift, sigma_base, sigma_full) -> dict:
    """Integer scales/offsets so that outputs spread over [0,127]:
    q_mul = round(2^S * 64/sigma * u), u ~ U(0.5,1.5); q_off = round(2^S * v), v ~ U(-8,8)."""
    g = rng(key, "q")
    two_s = float(1 << shift)
    u1, u2 = g.uniform(0.5, 1.5, c_out), g.uniform(0.5, 1.5, c_out)
    v1, v2 = g.uniform(-8, 8, c_out), g.uniform(-8, 8, c_out)
    return {
        "q_mul_base": np.clip(np.rint(two_s * 64.0 / sigma_base * u1), 1, 2**31 - 1).astype(np.int32),
        "q_mul_full": np.clip(np.rint(two_s * 64.0 / sigma_full * u2), 1, 2**31 - 1).astype(np.int32),
        "q_off_base": np.rint(two_s * v1).astype(np.int64),
        "q_off_full": np.rint(two_s * v2).astype(np.int64),
    }


# --------------------------------------------------------------------------- layer tables
@dataclass(frozen=True)
class LayerShape:
    name: str
    n: int
    hw: int
    c_in: int
    c_out: int
    stride: int = 1
    groups: int = 4


def cifar_resnet18_layers(batch=256, groups=4):
    """Gated 3x3 layers of a CIFAR-style ResNet-18 (c_in = c_out)."""
    return [LayerShape(f"c{c}@{hw}", batch, hw, c, c, 1, groups)
            for c, hw in ((64, 32), (128, 16), (256, 8), (512, 4))]


def imagenet_resnet18_layers(batch=64, groups=4, transitions=True):
    """Gated 3x3 layers of an ImageNet ResNet-18: four stride-1 shapes and the three
    stride-2 transitions between stages."""
    out = [LayerShape(f"c{c}@{hw}", batch, hw, c, c, 1, groups)
           for c, hw in ((64, 56), (128, 28), (256, 14), (512, 7))]
    if transitions:
        out += [LayerShape(f"c{c}to{2 * c}@{hw}s2", batch, hw, c, 2 * c, 2, groups)
                for c, hw in ((64, 56), (128, 28), (256, 14))]
    return out
