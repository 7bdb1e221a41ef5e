"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, and rejects bad descriptions before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_1805_12549_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols(header="cgconv.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cg_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = B.lib()
    names = _declared_symbols()
    assert set(B.EXPORTS) <= set(names)
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n


def test_library_exports_the_network_operators():
    lib = B.lib()
    names = _declared_symbols("cgnet.h")
    assert set(names) == set(B.NET_EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_network_operators_reject_bad_arguments_before_any_launch():
    lib = B.lib()
    buf = (C.c_uint8 * 4096)()
    base = C.addressof(buf)
    p = C.c_void_p((base + 15) & ~15)
    odd = C.c_void_p(p.value + 2)
    INVALID, ALIGN = 1, 3
    assert lib.cg_im2col_bf16(None, p, 1, 8, 8, 3, 7, 2, 3, 152, None) == INVALID
    assert lib.cg_im2col_bf16(p, p, 1, 8, 8, 3, 7, 2, 3, 144, None) == INVALID      # k_pad < 147
    assert lib.cg_im2col_bf16(p, p, 1, 8, 8, 3, 7, 2, 3, 150, None) == INVALID      # not a multiple of 8
    assert lib.cg_im2col_bf16(p, p, 1, 2, 2, 3, 7, 2, 0, 152, None) == INVALID      # filter larger than the image
    assert lib.cg_im2col_bf16(odd, p, 1, 8, 8, 3, 7, 2, 3, 152, None) == ALIGN
    assert lib.cg_subsample_bf16(p, p, 1, 8, 8, 12, 2, None) == INVALID             # channels not a multiple of 8
    assert lib.cg_subsample_bf16(p, odd, 1, 8, 8, 16, 2, None) == ALIGN
    assert lib.cg_maxpool_bf16(p, p, 1, 8, 8, 16, 3, 2, 3, None) == INVALID         # a window of padding only
    assert lib.cg_maxpool_bf16(p, None, 1, 8, 8, 16, 3, 2, 1, None) == INVALID
    assert lib.cg_avgpool_bf16(p, p, 0, 49, 16, None) == INVALID
    assert lib.cg_avgpool_bf16(odd, p, 1, 49, 16, None) == ALIGN


def test_status_strings():
    lib = B.lib()
    seen = {lib.cg_status_string(i) for i in range(8)}
    assert len(seen) == 8
    assert lib.cg_status_string(0) == b"ok"


def _desc(**kw):
    base = dict(n=2, h=8, w=8, c_in=16, c_out=16, kh=3, kw=3, stride=1, pad=1, groups=4,
                in_dtype=B.CG_F32, out_dtype=B.CG_F32, bn_eps=1e-5, relu=1, has_residual=0,
                requant_shift=0, algo=0, cond_mode=0, grouping=0)
    base.update(kw)
    return B.CgConvDesc(**base)


@pytest.mark.parametrize("kw", [dict(n=0), dict(c_in=15), dict(kh=3, kw=5), dict(groups=0),
                                dict(stride=0), dict(pad=-1), dict(in_dtype=7, out_dtype=7),
                                dict(out_dtype=B.CG_BF16), dict(h=1, w=1, pad=0),
                                dict(in_dtype=B.CG_I8, out_dtype=B.CG_I8, requant_shift=0),
                                dict(in_dtype=B.CG_I8, out_dtype=B.CG_I8, requant_shift=32),
                                dict(bn_eps=-1.0), dict(algo=9), dict(cond_mode=-1),
                                dict(grouping=2), dict(grouping=1, c_out=18),
                                dict(grouping=1, in_dtype=B.CG_I8, out_dtype=B.CG_I8,
                                     requant_shift=8)])
def test_create_rejects_bad_descriptions(kw):
    h = C.c_void_p()
    d = _desc(**kw)
    assert B.lib().cg_conv_create(C.byref(h), C.byref(d)) == 1      # CG_ERR_INVALID_ARG
    assert not h.value


def test_create_null_arguments():
    d = _desc()
    assert B.lib().cg_conv_create(None, C.byref(d)) == 1
    h = C.c_void_p()
    assert B.lib().cg_conv_create(C.byref(h), None) == 1


def test_tensor_algo_rejects_ineligible_layers():
    h = C.c_void_p()
    for kw in (dict(algo=B.CG_ALGO_TENSOR),                                  # fp32
               dict(algo=B.CG_ALGO_TENSOR, in_dtype=B.CG_BF16, out_dtype=B.CG_BF16, c_in=24,
                    c_out=16)):                                              # c_p = 6 channels
        d = _desc(**kw)
        assert B.lib().cg_conv_create(C.byref(h), C.byref(d)) == 2           # CG_ERR_UNSUPPORTED


def test_tap_stacked_algo_eligibility_is_decided_on_the_host():
    """CG_ALGO_TENSOR_STACKED: 3x3, stride 1, pad 1, bf16, 64 -> 64 channels, c_in/G a multiple of 16,
    width at most 128, no grouping, no channel-wise gate, no row compaction.  Layers outside report
    CG_ERR_UNSUPPORTED before any device is needed; a layer inside gets as far as the device."""
    import torch
    h = C.c_void_p()
    ok = dict(algo=B.CG_ALGO_TENSOR_STACKED, in_dtype=B.CG_BF16, out_dtype=B.CG_BF16, c_in=64, c_out=64,
              h=32, w=32, groups=4)
    for kw in (dict(w=129), dict(c_out=128), dict(c_in=128), dict(groups=8), dict(kh=1, kw=1, pad=0),
               dict(stride=2), dict(cond_mode=3), dict(channel_tau=0.5), dict(grouping=1),
               dict(in_dtype=B.CG_I8, out_dtype=B.CG_I8, requant_shift=8)):
        d = _desc(**{**ok, **kw})
        assert B.lib().cg_conv_create(C.byref(h), C.byref(d)) == 2, kw       # CG_ERR_UNSUPPORTED
    if not torch.cuda.is_available():
        for kw in (dict(), dict(w=56, h=56), dict(groups=1), dict(groups=2), dict(w=128, h=3)):
            d = _desc(**{**ok, **kw})
            assert B.lib().cg_conv_create(C.byref(h), C.byref(d)) == 5, kw   # CG_ERR_CUDA: eligible, no device


def test_null_handle_calls_are_safe():
    lib = B.lib()
    assert lib.cg_conv_workspace_bytes(None) == 0
    assert lib.cg_conv_host_staging_bytes(None) == 0
    assert lib.cg_conv_launches_per_forward(None) == 0
    assert lib.cg_conv_uses_tensor_cores(None) == 0
    lib.cg_conv_destroy(None)
    st = B.CgStats()
    assert lib.cg_conv_stats(None, C.byref(st), None) == 1
    bn = B.CgBnParams()
    assert lib.cg_conv_forward(None, None, None, None, C.byref(bn), None, None, None, None, None,
                               0, None) == 1


def test_create_without_a_device_reports_cuda_error():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = C.c_void_p()
    d = _desc()
    assert B.lib().cg_conv_create(C.byref(h), C.byref(d)) == 5               # CG_ERR_CUDA
    with pytest.raises(B.CgError):
        B.cg_conv_create(d)
