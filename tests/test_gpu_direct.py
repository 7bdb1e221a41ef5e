"""GPU parity of the CUDA-core direct path against the oracle: bit-exact masks and outputs,
because both run the sums in the order (r, s, c_in) with separately rounded multiply and add."""
import numpy as np
import pytest

from oracle import oracle as O
from tests import cases as K

pytestmark = pytest.mark.gpu

DIRECT = 1


@pytest.mark.parametrize("separate", [False, True])
def test_config1_fp32(separate):
    """2 x 16 x 8 x 8, G=4, Delta=0, fp32: shared and separate statistics."""
    s = O.Shape(2, 8, 8, 16, 16, groups=4)
    c = K.make_float_case(("cfg1", separate), s, "f32", delta=0.0, separate=separate, smooth=False)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=DIRECT)
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert 0.3 < st.density < 0.7
    assert st.executed_macs == st.gated_macs
    g.close()


@pytest.mark.parametrize("s", [
    O.Shape(1, 7, 9, 8, 5, groups=2),
    O.Shape(2, 9, 9, 12, 40, stride=2, groups=4),
    O.Shape(1, 6, 6, 6, 4, kh=1, kw=1, pad=0, groups=3),
    O.Shape(1, 8, 8, 4, 3, kh=5, kw=5, pad=2, groups=2),
    O.Shape(3, 5, 4, 8, 33, groups=1),
])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_odd_shapes(s, dtype):
    c = K.make_float_case("odd", s, dtype, density=0.4, residual=(s.c_out == 40))
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=DIRECT)
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    g.close()


@pytest.mark.parametrize("dv", [-K.INF, K.INF])
def test_delta_limits(dv):
    s = O.Shape(2, 8, 8, 16, 32, groups=4)
    c = K.make_float_case("lim", s, "bf16", delta=dv)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=DIRECT)
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert st.active == (st.outputs if dv < 0 else 0)
    g.close()


@pytest.mark.parametrize("s", [O.Shape(2, 7, 7, 12, 8, groups=4),
                               O.Shape(1, 9, 8, 64, 64, groups=4),
                               O.Shape(2, 8, 8, 32, 48, stride=2, groups=2)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_channel_grouping(s, dtype):
    """Section 3.3: output group i takes input group i as x_p and the other groups as x_r."""
    c = K.make_float_case("grp", s, dtype, density=0.4, grouped=True)
    ref = K.run_oracle(c)
    g = K.GpuCase(c)                       # AUTO must fall back to the direct kernels
    assert not g.conv.uses_tensor_cores
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    plain = K.run_oracle(K.make_float_case("grp", s, dtype, delta=c.delta))
    assert (plain.mask != ref.mask).any()  # grouping really changes the layer
    g.close()


def test_int8_bit_exact():
    s = O.Shape(2, 9, 9, 32, 48, groups=4)
    c = K.make_int8_case("i8", s, density=0.3)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=DIRECT)
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert 0.2 < st.density < 0.4
    assert len(np.unique(y)) > 16
    g.close()


def test_mask_optional_and_counters_accumulate():
    s = O.Shape(2, 8, 8, 16, 16, groups=4)
    c = K.make_float_case("acc", s, "bf16", density=0.3)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=DIRECT)
    y, _, st = g.run(with_mask=False)
    np.testing.assert_array_equal(y.view(np.uint32), ref.y.view(np.uint32))
    assert (g.mask.cpu().numpy() == -1).all()          # untouched
    for _ in range(3):
        g.conv.forward(g.x, g.wb, g.wc, g.bn, g.delta, g.y, g.mask, g.res)
    st = g.conv.stats()
    assert st.calls == 3 and st.active == 3 * ref.active and st.outputs == 3 * ref.outputs
    assert g.conv.stats().calls == 0                   # cleared by the read
    g.close()


def test_partial_sums_and_forward_host():
    import torch
    from paper_1805_12549_b200 import binding as B
    s = O.Shape(2, 8, 8, 16, 16, groups=4)
    c = K.make_float_case("host", s, "bf16", density=0.5)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=DIRECT)
    p = torch.empty((s.m, s.c_out), dtype=torch.float32, device="cuda")
    B.cg_conv_partial_sums(g.conv.handle, g.x, g.wb, p)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(p.cpu().numpy().reshape(ref.p.shape), ref.p)
    xh = g.x.cpu().pin_memory()
    yh = torch.empty(g.y.shape, dtype=g.y.dtype).pin_memory()
    mh = torch.empty(g.mask.shape, dtype=torch.int32).pin_memory()
    staging = torch.empty(B.cg_conv_host_staging_bytes(g.conv.handle), dtype=torch.uint8,
                          device="cuda")
    B.cg_conv_forward_host(g.conv.handle, xh, g.wb, g.wc, g.bn, g.delta, None, yh, mh, staging)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(yh.float().numpy().view(np.uint32), ref.y.view(np.uint32))
    np.testing.assert_array_equal(mh.numpy().view(np.uint32), ref.mask)
    g.close()


def test_forward_argument_errors():
    import ctypes as C
    import torch
    from paper_1805_12549_b200 import binding as B
    s = O.Shape(2, 8, 8, 16, 16, groups=4)
    c = K.make_float_case("err", s, "bf16", density=0.5)
    g = K.GpuCase(c, algo=DIRECT)
    lib, h = B.lib(), g.conv.handle
    sp = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = lambda **kw: [h, kw.get("x", g.x.data_ptr()), g.wb.data_ptr(), g.wc.data_ptr(),
                         C.byref(kw.get("bn", g.bn)), kw.get("delta", g.delta.data_ptr()),
                         kw.get("res", None), g.y.data_ptr(), g.mask.data_ptr(), None, 0, sp]
    assert lib.cg_conv_forward(*args()) == 0
    assert lib.cg_conv_forward(*args(x=None)) == 1
    assert lib.cg_conv_forward(*args(x=g.x.data_ptr() + 2)) == 3
    assert lib.cg_conv_forward(*args(delta=None)) == 1
    assert lib.cg_conv_forward(*args(res=g.y.data_ptr())) == 1
    bad = B.make_bn({k: v for k, v in g.params.items() if k != "gamma"})
    assert lib.cg_conv_forward(*args(bn=bad)) == 1
    g.conv.stats()
    g.close()


# ----------------------------------------------------------------------------- channel-wise gate
CHANNEL_GATE_SHAPES = [
    O.Shape(2, 8, 8, 16, 16, groups=4),
    O.Shape(3, 7, 9, 8, 40, groups=2),
    O.Shape(5, 14, 14, 64, 96, groups=4),
    O.Shape(2, 9, 9, 12, 33, stride=2, groups=4),
]


@pytest.mark.parametrize("s", CHANNEL_GATE_SHAPES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("tau", [0.3, 0.45])
def test_channel_wise_gate(s, dtype, tau):
    """Eq. 4 through the C ABI: per image, channels whose gate fires at fewer than tau_c*h'*w'
    positions take the base path everywhere.  Integer counts and one fp32 comparison, so the
    decisions, masks and outputs are bit-exact against the oracle."""
    c = K.make_float_case("chgate", s, dtype, density=0.4)
    c.channel_tau = tau
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=1)    # the direct kernels
    assert not g.conv.uses_tensor_cores
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert st.channels == ref.channels == s.n * s.c_out
    assert st.channels_skipped == ref.channels_skipped
    assert st.active == ref.active
    assert 0 < st.channels_skipped < st.channels, "the case should drop some channels, not all"
    # a second call reuses the workspace (counts are cleared per call)
    y2, mask2, st2 = g.run()
    np.testing.assert_array_equal(mask, mask2)
    assert st2.channels_skipped == ref.channels_skipped
    g.close()


def test_channel_wise_gate_limits_and_rejections():
    from paper_1805_12549_b200 import binding as B
    s = O.Shape(2, 8, 8, 16, 32, groups=4)
    c = K.make_float_case("chlim", s, "bf16", density=0.4)
    plain = K.run_oracle(c)
    c.channel_tau = 1.5                       # no count reaches 1.5*h'*w': every channel off
    ref = K.run_oracle(c)
    g = K.GpuCase(c)
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert st.active == 0 and st.channels_skipped == st.channels
    g.close()
    assert plain.active > 0
    # the channel-major kernel and int8 layers do not take the channel-wise gate
    with pytest.raises(B.CgError) as e:
        B.GatedConv(2, 28, 28, 128, 128, algo=B.CG_ALGO_TENSOR_CHANNELS, channel_tau=0.2)
    assert e.value.status == 2
    with pytest.raises(B.CgError) as e:
        B.GatedConv(2, 28, 28, 128, 128, dtype=B.CG_I8, requant_shift=8, channel_tau=0.2)
    assert e.value.status == 1
    with pytest.raises(B.CgError) as e:
        B.GatedConv(2, 8, 8, 16, 16, channel_tau=-0.1)
    assert e.value.status == 1


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_two_sided_gate_on_the_direct_path(dtype):
    """Section 3.2 through the C ABI: upper thresholds in cg_bn_params.delta_high; bit-exact."""
    s = O.Shape(2, 9, 10, 12, 40, groups=4)
    c = K.make_float_case("band", s, dtype, density=0.5)
    one_sided = K.run_oracle(c)
    c.delta_high = (c.delta + np.float32(0.8)).astype(np.float32)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=1)
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert 0 < ref.active < one_sided.active and st.active == ref.active
    g.close()
