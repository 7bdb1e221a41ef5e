"""Thin ctypes binding of the cgconv C ABI (include/cgconv.h).

Argument marshalling only: every step of the layer runs in the CUDA library.  Tensors are
torch CUDA tensors (device memory and streams are torch's); their data pointers go straight
through.  There is no CPU fallback: if the library cannot be loaded, importing fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

CG_OK = 0
CG_F32, CG_BF16, CG_I8 = 0, 1, 2
CG_ALGO_AUTO, CG_ALGO_DIRECT, CG_ALGO_TENSOR, CG_ALGO_TENSOR_ROWS, CG_ALGO_TENSOR_CHANNELS = 0, 1, 2, 3, 4
CG_ALGO_TENSOR_STACKED = 5
CG_KERNEL_DIRECT, CG_KERNEL_TENSOR_PIXEL_MAJOR, CG_KERNEL_TENSOR_CHANNEL_MAJOR = 0, 1, 2
CG_KERNEL_TENSOR_TAP_STACKED = 3
CG_COND_AUTO, CG_COND_DENSE, CG_COND_SKIP_TILES, CG_COND_COMPACT = 0, 1, 2, 3

EXPORTS = ("cg_conv_create", "cg_conv_workspace_bytes", "cg_conv_forward",
           "cg_conv_host_staging_bytes", "cg_conv_forward_host", "cg_conv_partial_sums",
           "cg_conv_stats", "cg_conv_launches_per_forward", "cg_conv_uses_tensor_cores",
           "cg_conv_kernel_id", "cg_conv_plan_string", "cg_conv_destroy", "cg_status_string", "cg_conv_forward_static")
# include/cgnet.h: the ungated operators of a whole network
NET_EXPORTS = ("cg_im2col_bf16", "cg_subsample_bf16", "cg_maxpool_bf16", "cg_avgpool_bf16")


class CgConvDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n", "h", "w", "c_in", "c_out", "kh", "kw", "stride",
                                         "pad", "groups", "in_dtype", "out_dtype")] + \
               [("bn_eps", C.c_float)] + \
               [(k, C.c_int32) for k in ("relu", "has_residual", "requant_shift", "algo",
                                         "cond_mode", "grouping")] + \
               [("channel_tau", C.c_float)]


class CgBnParams(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("gamma", "beta", "mean_base", "var_base", "mean_full",
                                          "var_full", "gate_mean", "gate_var", "q_gate_thr",
                                          "q_mul_base", "q_mul_full", "q_off_base", "q_off_full",
                                          "delta_high")]


class CgStats(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("calls", "outputs", "active", "dense_macs", "gated_macs",
                                         "executed_macs", "tiles_total", "tiles_skipped",
                                         "rows_total", "rows_active")] + \
               [("device_status", C.c_int32), ("device_site", C.c_int32)] + \
               [("channels", C.c_int64), ("channels_skipped", C.c_int64)]


_lib = None


def lib():
    """Load libcgconv.so (building it first if the sources are newer)."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.cg_conv_create.restype = C.c_int
        L.cg_conv_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(CgConvDesc)]
        L.cg_conv_workspace_bytes.restype = C.c_size_t
        L.cg_conv_workspace_bytes.argtypes = [C.c_void_p]
        L.cg_conv_forward.restype = C.c_int
        L.cg_conv_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.POINTER(CgBnParams), C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.cg_conv_host_staging_bytes.restype = C.c_size_t
        L.cg_conv_host_staging_bytes.argtypes = [C.c_void_p]
        L.cg_conv_forward_host.restype = C.c_int
        L.cg_conv_forward_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.POINTER(CgBnParams), C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                           C.c_void_p]
        L.cg_conv_partial_sums.restype = C.c_int
        L.cg_conv_partial_sums.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p]
        L.cg_conv_stats.restype = C.c_int
        L.cg_conv_stats.argtypes = [C.c_void_p, C.POINTER(CgStats), C.c_void_p]
        L.cg_conv_launches_per_forward.restype = C.c_int
        L.cg_conv_launches_per_forward.argtypes = [C.c_void_p]
        L.cg_conv_uses_tensor_cores.restype = C.c_int
        L.cg_conv_uses_tensor_cores.argtypes = [C.c_void_p]
        L.cg_conv_kernel_id.restype = C.c_int
        L.cg_conv_kernel_id.argtypes = [C.c_void_p]
        L.cg_conv_plan_string.restype = C.c_int
        L.cg_conv_plan_string.argtypes = [C.c_void_p, C.c_char_p, C.c_size_t]
        L.cg_conv_destroy.restype = None
        L.cg_conv_destroy.argtypes = [C.c_void_p]
        L.cg_conv_forward_static.restype = C.c_int
        L.cg_conv_forward_static.argtypes = [C.POINTER(CgConvDesc), C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.POINTER(CgBnParams), C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.POINTER(CgStats), C.c_void_p]
        L.cg_status_string.restype = C.c_char_p
        L.cg_status_string.argtypes = [C.c_int]
        i = C.c_int
        L.cg_im2col_bf16.restype = C.c_int
        L.cg_im2col_bf16.argtypes = [C.c_void_p, C.c_void_p, i, i, i, i, i, i, i, i, C.c_void_p]
        L.cg_subsample_bf16.restype = C.c_int
        L.cg_subsample_bf16.argtypes = [C.c_void_p, C.c_void_p, i, i, i, i, i, C.c_void_p]
        L.cg_maxpool_bf16.restype = C.c_int
        L.cg_maxpool_bf16.argtypes = [C.c_void_p, C.c_void_p, i, i, i, i, i, i, i, C.c_void_p]
        L.cg_avgpool_bf16.restype = C.c_int
        L.cg_avgpool_bf16.argtypes = [C.c_void_p, C.c_void_p, i, i, i, C.c_void_p]
        _lib = L
    return _lib


class CgError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().cg_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != CG_OK:
        raise CgError(status, where)


_TORCH_DTYPE = {CG_F32: torch.float32, CG_BF16: torch.bfloat16, CG_I8: torch.int8}


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


@dataclass
class Stats:
    calls: int
    outputs: int
    active: int
    dense_macs: int
    gated_macs: int
    executed_macs: int
    tiles_total: int
    tiles_skipped: int
    rows_total: int
    rows_active: int
    device_status: int
    device_site: int
    channels: int = 0
    channels_skipped: int = 0

    @property
    def density(self):
        return self.active / max(self.outputs, 1)


def cg_conv_create(desc: CgConvDesc) -> C.c_void_p:
    h = C.c_void_p()
    _check(lib().cg_conv_create(C.byref(h), C.byref(desc)), "cg_conv_create")
    return h


def cg_conv_destroy(h):
    lib().cg_conv_destroy(h)


def cg_conv_workspace_bytes(h) -> int:
    return int(lib().cg_conv_workspace_bytes(h))


def make_bn(params: dict) -> CgBnParams:
    """dict of torch CUDA tensors (missing/None -> NULL) -> cg_bn_params."""
    bn = CgBnParams()
    for k, _ in CgBnParams._fields_:
        t = params.get(k)
        setattr(bn, k, None if t is None else t.data_ptr())
    return bn


def cg_conv_forward(h, x, w_base, w_cond, bn: CgBnParams, delta, residual, y, mask_out,
                    workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().cg_conv_forward(h, _ptr(x), _ptr(w_base), _ptr(w_cond), C.byref(bn), _ptr(delta),
                                 _ptr(residual), _ptr(y), _ptr(mask_out), _ptr(workspace),
                                 ws_bytes, _stream_ptr(stream)), "cg_conv_forward")


def cg_conv_host_staging_bytes(h) -> int:
    return int(lib().cg_conv_host_staging_bytes(h))


def cg_conv_forward_host(h, x_host, w_base, w_cond, bn: CgBnParams, delta, residual_host, y_host,
                         mask_host, staging, stream=None):
    _check(lib().cg_conv_forward_host(h, _ptr(x_host), _ptr(w_base), _ptr(w_cond), C.byref(bn),
                                      _ptr(delta), _ptr(residual_host), _ptr(y_host),
                                      _ptr(mask_host), _ptr(staging),
                                      staging.numel() * staging.element_size(),
                                      _stream_ptr(stream)), "cg_conv_forward_host")


def cg_conv_partial_sums(h, x, w_base, p_out, stream=None):
    _check(lib().cg_conv_partial_sums(h, _ptr(x), _ptr(w_base), _ptr(p_out), _stream_ptr(stream)),
           "cg_conv_partial_sums")


def cg_conv_stats(h, stream=None, check=True) -> Stats:
    st = CgStats()
    rc = lib().cg_conv_stats(h, C.byref(st), _stream_ptr(stream))
    out = Stats(*[getattr(st, k) for k, _ in CgStats._fields_])
    if check:
        _check(rc, f"cg_conv_stats (device site {out.device_site})")
    return out


CG_STATIC_MAX_C_OUT = 2048


def cg_conv_forward_static(desc: CgConvDesc, x, w_base, w_cond, bn: CgBnParams, delta, residual, y,
                           mask_out, want_stats=False, stream=None):
    """The layer without a handle and without any allocation (see include/cgconv.h): scratch
    lives in a fixed array inside the library.  Calls on one device must not overlap."""
    st = CgStats() if want_stats else None
    _check(lib().cg_conv_forward_static(C.byref(desc), _ptr(x), _ptr(w_base), _ptr(w_cond),
                                        C.byref(bn), _ptr(delta), _ptr(residual), _ptr(y),
                                        _ptr(mask_out), C.byref(st) if st is not None else None,
                                        _stream_ptr(stream)), "cg_conv_forward_static")
    return None if st is None else Stats(*[getattr(st, k) for k, _ in CgStats._fields_])


def cg_conv_launches_per_forward(h) -> int:
    return int(lib().cg_conv_launches_per_forward(h))


def cg_conv_uses_tensor_cores(h) -> bool:
    return bool(lib().cg_conv_uses_tensor_cores(h))


def cg_conv_kernel_id(h) -> int:
    return int(lib().cg_conv_kernel_id(h))


def cg_conv_plan_string(h) -> str:
    buf = C.create_string_buffer(512)
    lib().cg_conv_plan_string(h, buf, len(buf))
    return buf.value.decode()


def cg_im2col_bf16(x, a, k, stride, pad, stream=None):
    """x [n,h,w,c] -> a [n,h',w',k_pad] (include/cgnet.h)."""
    n, h, w, c = x.shape
    _check(lib().cg_im2col_bf16(_ptr(x), _ptr(a), n, h, w, c, k, stride, pad, a.shape[-1],
                                _stream_ptr(stream)), "cg_im2col_bf16")


def cg_subsample_bf16(x, y, stride, stream=None):
    n, h, w, c = x.shape
    _check(lib().cg_subsample_bf16(_ptr(x), _ptr(y), n, h, w, c, stride, _stream_ptr(stream)),
           "cg_subsample_bf16")


def cg_maxpool_bf16(x, y, k, stride, pad, stream=None):
    n, h, w, c = x.shape
    _check(lib().cg_maxpool_bf16(_ptr(x), _ptr(y), n, h, w, c, k, stride, pad, _stream_ptr(stream)),
           "cg_maxpool_bf16")


def cg_avgpool_bf16(x, y, stream=None):
    n, h, w, c = x.shape
    _check(lib().cg_avgpool_bf16(_ptr(x), _ptr(y), n, h * w, c, _stream_ptr(stream)), "cg_avgpool_bf16")


class GatedConv:
    """Convenience owner of one handle plus its workspace (still argument marshalling only)."""

    def __init__(self, n, h, w, c_in, c_out, *, k=3, stride=1, pad=1, groups=4, dtype=CG_BF16,
                 bn_eps=1e-5, relu=True, has_residual=False, requant_shift=0,
                 algo=CG_ALGO_AUTO, cond_mode=CG_COND_AUTO, grouping=False, channel_tau=0.0,
                 device="cuda"):
        self.desc = CgConvDesc(n, h, w, c_in, c_out, k, k, stride, pad, groups, dtype, dtype,
                               bn_eps, int(relu), int(has_residual), requant_shift, algo, cond_mode,
                               int(grouping), float(channel_tau))
        self.handle = cg_conv_create(self.desc)
        self.dtype = dtype
        self.ho = (h + 2 * pad - k) // stride + 1
        self.wo = (w + 2 * pad - k) // stride + 1
        self.m = n * self.ho * self.wo
        self.c_out = c_out
        self.words = (c_out + 31) // 32
        self.device = device
        nbytes = cg_conv_workspace_bytes(self.handle)
        self.workspace = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=device) \
            if nbytes else None

    def alloc_outputs(self):
        y = torch.empty((self.desc.n, self.ho, self.wo, self.c_out), dtype=_TORCH_DTYPE[self.dtype],
                        device=self.device)
        mask = torch.empty((self.m, self.words), dtype=torch.int32, device=self.device)
        return y, mask

    def forward(self, x, w_base, w_cond, bn: CgBnParams, delta, y, mask=None, residual=None,
                stream=None):
        cg_conv_forward(self.handle, x, w_base, w_cond, bn, delta, residual, y, mask,
                        self.workspace, stream)

    def stats(self, stream=None, check=True) -> Stats:
        return cg_conv_stats(self.handle, stream, check)

    @property
    def uses_tensor_cores(self):
        return cg_conv_uses_tensor_cores(self.handle)

    @property
    def kernel_id(self):
        return cg_conv_kernel_id(self.handle)

    @property
    def plan(self):
        return cg_conv_plan_string(self.handle)

    def close(self):
        if self.handle is not None:
            cg_conv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
