"""ctypes front end of the CPU oracle (cg_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA library never loads it, and it
never loads the CUDA library.

The functions mirror the layer of Channel Gating Neural Networks (Section 3.1,
Eq. 1-3, and the two batch norms of Section 4); see the header of
cg_oracle.cpp for the passage each step follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cg_oracle.cpp")
_LIB = os.path.join(_HERE, "libcgoracle.so")


def build(force: bool = False) -> str:
    """Compile cg_oracle.cpp with g++ (OpenMP, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-fPIC", "-shared", "-o", _LIB + ".tmp", _SRC]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


class _Desc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n", "h", "w", "c_in", "c_out", "kh", "kw", "stride", "pad",
                                         "groups")] + \
               [("bn_eps", C.c_float)] + \
               [(k, C.c_int32) for k in ("relu", "out_bf16", "acc_double", "gate_form", "grouped")] + \
               [("channel_tau", C.c_float), ("delta_high", C.c_void_p)]


class _Counts(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("outputs", "active", "base_macs", "cond_macs", "dense_macs",
                                         "channels", "channels_skipped")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.cgo_round_bf16.restype = C.c_float
        _lib.cgo_round_bf16.argtypes = [C.c_float]
        _lib.cgo_out_dim.restype = C.c_int
        _lib.cgo_num_threads.restype = C.c_int
    return _lib


@dataclass
class Shape:
    n: int
    h: int
    w: int
    c_in: int
    c_out: int
    kh: int = 3
    kw: int = 3
    stride: int = 1
    pad: int = 1
    groups: int = 4
    bn_eps: float = 1e-5
    relu: int = 1

    @property
    def ho(self):
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def wo(self):
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1

    @property
    def c_p(self):
        return self.c_in // self.groups

    @property
    def c_r(self):
        return self.c_in - self.c_p

    @property
    def m(self):
        return self.n * self.ho * self.wo

    @property
    def words(self):
        return (self.c_out + 31) // 32


@dataclass
class Result:
    y: np.ndarray            # [n, h', w', c_out]
    mask: np.ndarray         # uint32 [n*h'*w', ceil(c_out/32)]
    p: np.ndarray            # partial sums [n, h', w', c_out]
    outputs: int
    active: int
    base_macs: int
    cond_macs: int
    dense_macs: int
    channels: int = 0            # n * c_out
    channels_skipped: int = 0    # channels switched off by the channel-wise gate (Eq. 4)

    @property
    def density(self):
        return self.active / max(self.outputs, 1)

    @property
    def gated_macs(self):
        return self.base_macs + self.cond_macs


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def num_threads() -> int:
    return int(lib().cgo_num_threads())


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16, returned as float32 (the oracle's own rounding)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    f = lib().cgo_round_bf16
    flat_in, flat_out = a.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = f(float(flat_in[i]))
    return out


def fold_params(s: Shape, bn: dict, delta) -> dict:
    """Per-channel t, a1, b1, a2, b2 exactly as the oracle derives them."""
    d = _Desc(s.n, s.h, s.w, s.c_in, s.c_out, s.kh, s.kw, s.stride, s.pad, s.groups, s.bn_eps,
              s.relu, 0, 0, 0, 0, 0.0)
    arrs = {k: _f32(bn.get(k)) for k in ("gamma", "beta", "mean_base", "var_base", "mean_full",
                                        "var_full", "gate_mean", "gate_var")}
    delta = _f32(delta)
    out = {k: np.empty(s.c_out, np.float32) for k in ("t", "a1", "b1", "a2", "b2")}
    lib().cgo_fold_params(C.byref(d), *[_ptr(arrs[k], C.c_float) for k in
                                        ("gamma", "beta", "mean_base", "var_base", "mean_full",
                                         "var_full", "gate_mean", "gate_var")],
                          _ptr(delta, C.c_float), *[_ptr(out[k], C.c_float) for k in
                                                    ("t", "a1", "b1", "a2", "b2")])
    return out


def gated_conv(s: Shape, x, w_base, w_cond, bn: dict, delta, residual=None, *, out_bf16=False,
               acc_double=False, gate_form=0, grouped=False, channel_tau=0.0, delta_high=None) -> Result:
    """Floating-point gated layer.  bn holds gamma, beta, mean_base, var_base, mean_full,
    var_full and optionally gate_mean, gate_var (absent/None: BN1's statistics).
    channel_tau > 0 adds the channel-wise gate of Eq. 4."""
    d = _Desc(s.n, s.h, s.w, s.c_in, s.c_out, s.kh, s.kw, s.stride, s.pad, s.groups, s.bn_eps,
              s.relu, int(out_bf16), int(acc_double), int(gate_form), int(grouped),
              float(channel_tau), None)
    delta_high = _f32(delta_high)
    if delta_high is not None:
        assert delta_high.size == s.c_out
        d.delta_high = delta_high.ctypes.data     # two-sided gate of Section 3.2
    x = _f32(x)
    w_base = _f32(w_base)
    w_cond = _f32(w_cond)
    assert x.size == s.n * s.h * s.w * s.c_in
    assert w_base.size == s.c_out * s.kh * s.kw * s.c_p
    assert w_cond.size == s.c_out * s.kh * s.kw * s.c_r
    arrs = {k: _f32(bn.get(k)) for k in ("gamma", "beta", "mean_base", "var_base", "mean_full",
                                        "var_full", "gate_mean", "gate_var")}
    for k in ("gamma", "beta", "mean_base", "var_base", "mean_full", "var_full"):
        assert arrs[k] is not None and arrs[k].size == s.c_out, k
    delta = _f32(delta)
    assert delta.size == s.c_out
    residual = _f32(residual)
    y = np.empty((s.n, s.ho, s.wo, s.c_out), np.float32)
    mask = np.zeros((s.m, s.words), np.uint32)
    p = np.empty((s.n, s.ho, s.wo, s.c_out), np.float32)
    cnt = _Counts()
    rc = lib().cgo_gated_conv(
        C.byref(d), _ptr(x, C.c_float), _ptr(w_base, C.c_float), _ptr(w_cond, C.c_float),
        *[_ptr(arrs[k], C.c_float) for k in ("gamma", "beta", "mean_base", "var_base",
                                             "mean_full", "var_full", "gate_mean", "gate_var")],
        _ptr(delta, C.c_float), _ptr(residual, C.c_float), _ptr(y, C.c_float),
        _ptr(mask, C.c_uint32), _ptr(p, C.c_float), C.byref(cnt))
    if rc != 0:
        raise ValueError("oracle rejected the layer description")
    return Result(y, mask, p, cnt.outputs, cnt.active, cnt.base_macs, cnt.cond_macs, cnt.dense_macs,
                  cnt.channels, cnt.channels_skipped)


def gated_conv_i8(s: Shape, shift: int, x, w_base, w_cond, q: dict) -> Result:
    """Quantised gated layer.  q holds q_gate_thr, q_mul_base, q_mul_full (int32) and
    q_off_base, q_off_full (int64), one entry per output channel."""
    d = _Desc(s.n, s.h, s.w, s.c_in, s.c_out, s.kh, s.kw, s.stride, s.pad, s.groups, s.bn_eps,
              s.relu, 0, 0, 0, 0, 0.0)
    x = np.ascontiguousarray(x, dtype=np.int8)
    w_base = np.ascontiguousarray(w_base, dtype=np.int8)
    w_cond = np.ascontiguousarray(w_cond, dtype=np.int8)
    assert x.size == s.n * s.h * s.w * s.c_in
    assert w_base.size == s.c_out * s.kh * s.kw * s.c_p
    assert w_cond.size == s.c_out * s.kh * s.kw * s.c_r
    thr = np.ascontiguousarray(q["q_gate_thr"], dtype=np.int32)
    mb = np.ascontiguousarray(q["q_mul_base"], dtype=np.int32)
    mf = np.ascontiguousarray(q["q_mul_full"], dtype=np.int32)
    ob = np.ascontiguousarray(q["q_off_base"], dtype=np.int64)
    of = np.ascontiguousarray(q["q_off_full"], dtype=np.int64)
    y = np.empty((s.n, s.ho, s.wo, s.c_out), np.int8)
    mask = np.zeros((s.m, s.words), np.uint32)
    p = np.empty((s.n, s.ho, s.wo, s.c_out), np.int32)
    cnt = _Counts()
    rc = lib().cgo_gated_conv_i8(
        C.byref(d), C.c_int32(shift), _ptr(x, C.c_int8), _ptr(w_base, C.c_int8),
        _ptr(w_cond, C.c_int8), _ptr(thr, C.c_int32), _ptr(mb, C.c_int32), _ptr(mf, C.c_int32),
        _ptr(ob, C.c_int64), _ptr(of, C.c_int64), _ptr(y, C.c_int8), _ptr(mask, C.c_uint32),
        _ptr(p, C.c_int32), C.byref(cnt))
    if rc != 0:
        raise ValueError("oracle rejected the layer description")
    return Result(y, mask, p, cnt.outputs, cnt.active, cnt.base_macs, cnt.cond_macs, cnt.dense_macs)


def unpack_mask(mask: np.ndarray, c_out: int) -> np.ndarray:
    """uint32 words [m, ceil(c_out/32)] -> bool [m, c_out]."""
    bits = ((mask[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).astype(bool)
    return bits.reshape(mask.shape[0], -1)[:, :c_out]
