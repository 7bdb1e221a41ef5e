"""GPU parity of the channel-major tcgen05 kernel (output channels on the MMA's M side, pixels on
its N side) against the oracle.

bf16 bar: masks equal except where the oracle's normalised partial sum lies within 1e-3 of
Delta (that count is printed); outputs within 2e-2 + 1e-2*|ref| wherever the masks agree."""
import numpy as np
import pytest

from oracle import oracle as O
from tests import cases as K

pytestmark = pytest.mark.gpu

CHANNELS = 4     # CG_ALGO_TENSOR_CHANNELS
DENSE, SKIP = 1, 2

# (shape, why): several pixel tiles, ragged tails, one and several channel tiles, every K-stage layout
SHAPES = [
    (O.Shape(3, 28, 28, 128, 128, groups=4), "c_p = 32: base stages of two taps, chunk 0 shared by both paths"),
    (O.Shape(2, 56, 56, 64, 64, groups=4), "c_p = 16, 64 output channels: half of the M rows are padding"),
    (O.Shape(3, 14, 14, 256, 256, groups=4), "c_p = 64, two channel tiles"),
    (O.Shape(5, 7, 7, 512, 512, groups=4), "c_p = 128, four channel tiles, whole images per copy"),
    (O.Shape(2, 32, 32, 64, 64, groups=4), "CIFAR 32x32"),
    (O.Shape(2, 16, 16, 128, 128, groups=4), "CIFAR 16x16"),
    (O.Shape(3, 8, 8, 256, 256, groups=4), "8x8 images"),
    (O.Shape(7, 4, 4, 512, 512, groups=4), "4x4 images, ragged batch"),
    (O.Shape(2, 28, 28, 128, 128, groups=8), "G = 8, c_p = 16"),
    (O.Shape(2, 14, 14, 256, 64, groups=8), "G = 8, c_p = 32, c_out != c_in"),
    (O.Shape(2, 13, 11, 64, 192, groups=2), "odd extents, G = 2, second channel tile half full"),
    (O.Shape(2, 9, 9, 64, 64, kh=1, kw=1, pad=0, groups=4), "1x1 kernel: no padding rows or columns"),
    (O.Shape(2, 12, 12, 64, 96, kh=5, kw=5, pad=2, groups=2), "5x5 kernel, pad 2, 96 output channels"),
    (O.Shape(40, 28, 28, 128, 128, groups=4), "several jobs per CTA"),
    (O.Shape(256, 4, 4, 128, 128, groups=4), "many small images per pixel tile"),
    (O.Shape(3, 56, 56, 64, 64, groups=8), "G = 8 at 64 channels: c_p = 8, weights repacked into the workspace"),
    (O.Shape(2, 17, 9, 64, 128, groups=8), "c_p = 8, odd extents, 128 output channels"),
    (O.Shape(1, 6, 200, 64, 64, groups=4), "one image, 200 pixels wide: a sub-tile is a single row"),
    (O.Shape(1, 3, 3, 64, 32, groups=4), "one 3x3 image, 32 output channels: a single job"),
    (O.Shape(2, 10, 10, 512, 128, groups=2), "c_p = 256: four base chunks, 72 K stages"),
]


def _run(c, cond_mode=0, with_mask=True):
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=CHANNELS, cond_mode=cond_mode)
    assert g.conv.uses_tensor_cores and g.conv.kernel_id == 2, g.conv.plan
    y, mask, st = g.run(with_mask=with_mask)
    if not with_mask:
        mask = ref.mask        # nothing was written: compare the outputs only
    exempt = K.compare(c, ref, y, mask, st if with_mask else None)
    plan = g.conv.plan
    g.close()
    return ref, st, exempt, plan


@pytest.mark.parametrize("s,why", SHAPES, ids=[w for _, w in SHAPES])
def test_parity_at_30_percent(s, why):
    c = K.make_float_case("ch30", s, "bf16", density=0.3)
    ref, st, exempt, plan = _run(c)
    print(f"{why}: density {st.density:.3f}, near-tie mismatches {exempt}, {plan}")
    assert abs(st.density - ref.density) < 2e-3
    assert 0.2 < st.density < 0.4
    assert st.rows_total == s.m * s.words          # one mask word per pixel and 32 channels


@pytest.mark.parametrize("s,why", SHAPES[:4] + SHAPES[11:13], ids=[w for _, w in SHAPES[:4] + SHAPES[11:13]])
@pytest.mark.parametrize("dv", [-K.INF, K.INF])
def test_delta_limits(s, why, dv):
    """All gates open: the ordinary layer.  All gates shut: base path only, every sub-tile skips
    its conditional MMAs."""
    c = K.make_float_case("chlim", s, "bf16", delta=dv)
    ref, st, exempt, _ = _run(c)
    assert exempt == 0
    if dv < 0:
        assert st.active == st.outputs and st.tiles_skipped == 0
    else:
        assert st.active == 0 and st.tiles_skipped == st.tiles_total > 0


@pytest.mark.parametrize("s,why", SHAPES[:4], ids=[w for _, w in SHAPES[:4]])
def test_dense_mode_matches_skip_mode(s, why):
    c = K.make_float_case("chdense", s, "bf16", density=0.1, rho=0.7)
    ref, st_d, _, _ = _run(c, cond_mode=DENSE)
    _, st_s, _, _ = _run(c, cond_mode=SKIP)
    assert st_d.active == st_s.active
    assert st_d.tiles_skipped == 0
    assert st_s.executed_macs <= st_d.executed_macs


def test_idle_sub_tiles_are_skipped():
    """Blank images give P = 0 below every (positive) threshold: the sub-tiles that lie wholly
    inside them issue no conditional MMAs."""
    s = O.Shape(8, 28, 28, 128, 128, groups=4)
    c = K.make_float_case("chskip", s, "bf16", density=0.05, rho=0.9)
    c.x[2:6] = 0.0
    t = O.fold_params(s, c.bn, c.delta)["t"]
    assert (t > 0).all()
    ref, st, _, plan = _run(c, cond_mode=SKIP)
    print(plan, st.tiles_skipped, st.tiles_total)
    assert st.tiles_skipped > 0
    assert st.rows_active < st.rows_total


def test_ungated_layer_groups_1():
    """G = 1: the base path is the whole convolution, there is no conditional path; the gate is
    still evaluated and selects between the two batch norms."""
    for s in (O.Shape(3, 14, 14, 128, 128, groups=1), O.Shape(2, 9, 9, 64, 256, kh=1, kw=1, pad=0, groups=1)):
        c = K.make_float_case("chg1", s, "bf16", density=0.3)
        ref, st, exempt, _ = _run(c)
        assert st.gated_macs == st.dense_macs
        assert abs(st.density - ref.density) < 2e-3


def test_identity_activation():
    s = O.Shape(3, 14, 14, 128, 128, groups=4, relu=0)
    c = K.make_float_case("chnorelu", s, "bf16", density=0.3)
    ref, st, exempt, _ = _run(c)
    assert (ref.y < 0).any()


def test_mask_pointer_may_be_null():
    s = O.Shape(3, 14, 14, 128, 128, groups=4)
    c = K.make_float_case("chnomask", s, "bf16", density=0.3)
    _run(c, with_mask=False)


def test_nan_input_does_not_fire():
    """A NaN partial sum compares false (gate shut) and the ReLU maps NaN to 0, as in the oracle."""
    s = O.Shape(2, 14, 14, 128, 128, groups=4)
    c = K.make_float_case("chnan", s, "bf16", density=0.3)
    c.x[0, 5, 5, 3] = np.nan          # a base-path channel: every output around (5,5) of image 0
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=CHANNELS)
    y, mask, st = g.run()
    g.close()
    d_ref = O.unpack_mask(ref.mask, s.c_out)
    d_gpu = O.unpack_mask(mask, s.c_out)
    nan_rows = np.isnan(ref.p.reshape(-1, s.c_out)).any(axis=1)
    assert nan_rows.sum() == 9
    assert not d_gpu[nan_rows].any() and not d_ref[nan_rows].any()
    yr = y.reshape(-1, s.c_out)
    assert (yr[nan_rows] == 0).all() and (ref.y.reshape(-1, s.c_out)[nan_rows] == 0).all()
    ok = ~nan_rows
    np.testing.assert_array_equal(d_gpu[ok], d_ref[ok])


RESIDUAL_SHAPES = [
    (O.Shape(3, 28, 28, 128, 128, groups=4), "one channel tile"),
    (O.Shape(7, 4, 4, 512, 512, groups=4), "small images, four channel tiles"),
]


@pytest.mark.parametrize("s,why", RESIDUAL_SHAPES, ids=[w for _, w in RESIDUAL_SHAPES])
def test_residual_input(s, why):
    c = K.make_float_case("chres", s, "bf16", density=0.3, residual=True)
    ref, st, exempt, _ = _run(c)
    assert abs(st.density - ref.density) < 2e-3


def test_two_calls_accumulate_and_are_deterministic():
    s = O.Shape(2, 28, 28, 128, 128, groups=4)
    c = K.make_float_case("chdet", s, "bf16", density=0.3)
    g = K.GpuCase(c, algo=CHANNELS)
    y1, m1, st1 = g.run()
    y2, m2, st2 = g.run()
    np.testing.assert_array_equal(y1.view(np.uint32), y2.view(np.uint32))
    np.testing.assert_array_equal(m1, m2)
    assert st1.active == st2.active and st1.calls == st2.calls == 1
    g.close()


@pytest.mark.parametrize("workload,layer", [
    ("imagenet", "c128@28"), ("imagenet", "c256@14"), ("imagenet", "c512@7"),
    ("cifar", "c128@16"), ("cifar", "c256@8"), ("cifar", "c512@4")])
def test_full_size_layers_on_sampled_images(workload, layer):
    """The layer shapes of the two benchmark workloads at benchmark batch; images are independent,
    so the oracle checks a sample of them one by one."""
    from paper_1805_12549_b200 import synth
    layers = synth.imagenet_resnet18_layers(64, 4) if workload == "imagenet" else synth.cifar_resnet18_layers(256, 4)
    ls = {l.name: l for l in layers}[layer]
    s = O.Shape(ls.n, ls.hw, ls.hw, ls.c_in, ls.c_out, stride=ls.stride, groups=4)
    c = K.make_float_case("chfull", s, "bf16", density=0.3, calib_images=2)
    g = K.GpuCase(c, algo=CHANNELS)
    assert g.conv.kernel_id == 2
    y, mask, st = g.run()
    g.close()
    assert abs(st.density - 0.3) < 0.04
    words = s.words
    per_img = s.ho * s.wo
    for n in sorted({0, s.n // 4 + 1, (5 * s.n) // 8, s.n - 1}):
        s1 = O.Shape(**{**s.__dict__, "n": 1})
        c1 = K.Case(c.name, s1, c.dtype, c.x[n:n + 1], c.wb, c.wc, c.bn, c.delta)
        ref = K.run_oracle(c1)
        K.compare(c1, ref, y[n:n + 1], mask[n * per_img:(n + 1) * per_img].reshape(-1, words), None)


def test_default_choice_of_tensor_kernel():
    """CG_ALGO_TENSOR picks the channel-major kernel for 128 output channels, the tap-stacked kernel for
    64 -> 64 channel 3x3 layers whose width divides 32 and the pixel-major kernel elsewhere."""
    from paper_1805_12549_b200 import binding as B
    for shape, want in (((4, 28, 28, 128, 128, 1), 2), ((4, 56, 56, 64, 64, 1), 1), ((4, 32, 32, 64, 64, 1), 3), ((4, 28, 28, 128, 256, 2), 1)):
        n, h, w, ci, co, st = shape
        conv = B.GatedConv(n, h, w, ci, co, k=3, stride=st, pad=1, groups=4, dtype=B.CG_BF16, algo=B.CG_ALGO_TENSOR)
        assert conv.kernel_id == want, conv.plan
        conv.close()


GROUPED = [
    (O.Shape(5, 7, 7, 512, 512, groups=4), "512 channels, G = 4: one 128-channel tile per output group"),
    (O.Shape(3, 8, 8, 256, 256, groups=2), "256 channels, G = 2"),
    (O.Shape(2, 14, 14, 256, 512, groups=4), "c_out != c_in"),
]


@pytest.mark.parametrize("s,why", GROUPED, ids=[w for _, w in GROUPED])
def test_channel_grouping(s, why):
    """Section 3.3: output group i takes input group i as its base path and the other groups, in
    ascending order, as its conditional path."""
    c = K.make_float_case("tc2grp", s, "bf16", density=0.3, grouped=True)
    ref, st, exempt, _ = _run(c)
    assert abs(st.density - ref.density) < 2e-3 and 0.2 < st.density < 0.4


TWO_SIDED = [
    (O.Shape(3, 28, 28, 128, 128, groups=4), "128@28"),
    (O.Shape(3, 14, 14, 256, 256, groups=4), "256@14"),
    (O.Shape(3, 8, 8, 256, 256, groups=4), "256@8"),
]


@pytest.mark.parametrize("s,why", TWO_SIDED, ids=[w for _, w in TWO_SIDED])
def test_two_sided_gate(s, why):
    """Section 3.2: with upper thresholds the gate fires only between Delta_l and Delta_h."""
    c = K.make_float_case("band", s, "bf16", density=0.5)
    one_sided = K.run_oracle(c)
    c.delta_high = (c.delta + np.float32(0.8)).astype(np.float32)
    ref, st, exempt, _ = _run(c)
    assert 0 < ref.active < one_sided.active
    assert st.active == ref.active or exempt > 0
