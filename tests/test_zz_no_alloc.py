"""cg_conv_forward_static: the layer for callers that cannot allocate device memory (a host
that owns the whole device through its own pool, a loop that must not make synchronising
calls, a plug-in with no allocator).  It takes no handle and keeps its scratch in a fixed
array inside the library, so every call shares that scratch: the test calls it twice in a row
and checks both results against the regular entry point, which must match bit for bit because
both run the same direct-convolution arithmetic."""
import ctypes as C

import numpy as np
import pytest

from oracle import oracle as O
from tests import cases as K

pytestmark = pytest.mark.gpu


def _run_static(g, want_stats):
    import torch
    from paper_1805_12549_b200 import binding as B
    y = torch.full_like(g.y, 7.0)
    mask = torch.full_like(g.mask, -1)
    st = B.cg_conv_forward_static(g.conv.desc, g.x, g.wb, g.wc, g.bn, g.delta, g.res, y, mask,
                                  want_stats=want_stats)
    torch.cuda.synchronize()
    return y.float().cpu().numpy(), mask.cpu().numpy().view(np.uint32), st


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_entry_matches_regular_entry_twice(dtype):
    s1 = O.Shape(3, 14, 14, 64, 96, groups=4)
    s2 = O.Shape(2, 9, 11, 32, 40, stride=2, groups=2)
    for s, density in ((s1, 0.3), (s2, 0.6)):        # two calls in a row, different layers
        c = K.make_float_case(("static", dtype), s, dtype, density=density,
                              residual=(s is s2))
        g = K.GpuCase(c, algo=1)                     # regular entry point, direct kernels
        y_ref, mask_ref, st_ref = g.run()
        y, mask, st = _run_static(g, want_stats=True)
        np.testing.assert_array_equal(mask, mask_ref)
        np.testing.assert_array_equal(y.view(np.uint32), y_ref.view(np.uint32))
        assert st.active == st_ref.active and st.outputs == st_ref.outputs
        assert st.gated_macs == st_ref.gated_macs
        # and again on the same layer: the scratch left by the previous call must not leak in
        y2, mask2, st2 = _run_static(g, want_stats=True)
        np.testing.assert_array_equal(mask2, mask_ref)
        np.testing.assert_array_equal(y2.view(np.uint32), y_ref.view(np.uint32))
        assert st2.active == st_ref.active
        # against the oracle as well
        ref = K.run_oracle(c)
        K.compare(c, ref, y2, mask2, None, exact=True)
        g.close()


def test_static_entry_rejects_what_does_not_fit():
    import torch
    from paper_1805_12549_b200 import binding as B
    lib = B.lib()
    d = B.CgConvDesc(1, 4, 4, 16, B.CG_STATIC_MAX_C_OUT + 32, 3, 3, 1, 1, 4, B.CG_BF16, B.CG_BF16,
                     1e-5, 1, 0, 0, 0, 0)
    buf = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    bn = B.make_bn({k: buf for k in ("gamma", "beta", "mean_base", "var_base", "mean_full",
                                     "var_full")})
    p = C.c_void_p(buf.data_ptr())
    args = [C.byref(d), p, p, p, C.byref(bn), p, None, p, None, None, None]
    assert lib.cg_conv_forward_static(*args) == 4                    # CG_ERR_WORKSPACE
    d.c_out = 64
    d.in_dtype = d.out_dtype = B.CG_I8
    assert lib.cg_conv_forward_static(*args) == 2                    # CG_ERR_UNSUPPORTED
    d.in_dtype = d.out_dtype = B.CG_BF16
    args[1] = None
    assert lib.cg_conv_forward_static(*args) == 1                    # CG_ERR_INVALID_ARG
    torch.cuda.synchronize()
