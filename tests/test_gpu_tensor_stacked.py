"""GPU parity of the tap-stacked tcgen05 kernel (64 -> 64 channel 3x3 layers: the three taps of a
filter row share one MMA, the epilogue adds the neighbours' partial sums) against the oracle.

bf16 bar: masks equal except where the oracle's normalised partial sum lies within 1e-3 of
Delta (that count is printed); outputs within 2e-2 + 1e-2*|ref| wherever the masks agree."""
import numpy as np
import pytest

from oracle import oracle as O
from tests import cases as K

pytestmark = pytest.mark.gpu

STACKED = 5      # CG_ALGO_TENSOR_STACKED
DENSE, SKIP = 1, 2

SHAPES = [
    (O.Shape(2, 32, 32, 64, 64, groups=2), "32x32, G = 2: a warp is one image row"),
    (O.Shape(3, 32, 32, 64, 64, groups=4), "32x32, G = 4: one base K step, three conditional ones"),
    (O.Shape(2, 16, 16, 64, 64, groups=2), "16x16: two image rows per warp, eight per job"),
    (O.Shape(5, 8, 8, 64, 64, groups=4), "8x8: the job's box is taller than the image"),
    (O.Shape(2, 13, 32, 64, 64, groups=2), "13 rows: the last job of an image is ragged"),
    (O.Shape(3, 40, 16, 64, 64, groups=4), "40x16: five jobs per image"),
    (O.Shape(1, 1, 8, 64, 64, groups=2), "a single image row of 8 pixels"),
    (O.Shape(40, 32, 32, 64, 64, groups=2), "several jobs per CTA"),
    (O.Shape(2, 32, 32, 64, 64, groups=4, relu=0), "identity activation"),
    (O.Shape(2, 56, 56, 64, 64, groups=4), "56x56: two rows per job, row ends inside warps, neighbours across warps"),
    (O.Shape(2, 28, 28, 64, 64, groups=2), "28x28: four rows per job, 112 of 128 slots"),
    (O.Shape(3, 14, 14, 64, 64, groups=4), "14x14: nine rows per job, the image is two ragged jobs"),
    (O.Shape(3, 7, 7, 64, 64, groups=2), "7x7: the job's box is taller than the image"),
    (O.Shape(2, 9, 13, 64, 64, groups=4), "9x13: odd extents"),
    (O.Shape(1, 5, 64, 64, 64, groups=4), "64 wide: two full rows per job, 5 rows"),
    (O.Shape(1, 3, 128, 64, 64, groups=2), "128 wide: one row per job, two patch buffers"),
    (O.Shape(1, 4, 100, 64, 64, groups=4), "100 wide: one row per job, 28 idle slots"),
    (O.Shape(2, 6, 33, 64, 64, groups=4), "33 wide: every warp boundary falls inside a row"),
]
WIDE = [x for x in SHAPES if x[0].w in (56, 14, 33)]


def _run(c, cond_mode=0, with_mask=True):
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=STACKED, cond_mode=cond_mode)
    assert g.conv.uses_tensor_cores and g.conv.kernel_id == 3, g.conv.plan
    y, mask, st = g.run(with_mask=with_mask)
    if not with_mask:
        mask = ref.mask        # nothing was written: compare the outputs only
    exempt = K.compare(c, ref, y, mask, st if with_mask else None)
    plan = g.conv.plan
    g.close()
    return ref, st, exempt, plan


@pytest.mark.parametrize("s,why", SHAPES, ids=[w for _, w in SHAPES])
def test_parity_at_30_percent(s, why):
    c = K.make_float_case("st30", s, "bf16", density=0.3)
    ref, st, exempt, plan = _run(c)
    print(f"{why}: density {st.density:.3f}, near-tie mismatches {exempt}, {plan}")
    assert abs(st.density - ref.density) < 2e-3
    assert 0.2 < st.density < 0.4
    assert st.rows_total == s.m
    if not s.relu:
        assert (ref.y < 0).any()


@pytest.mark.parametrize("s,why", SHAPES[:6] + WIDE, ids=[w for _, w in SHAPES[:6] + WIDE])
@pytest.mark.parametrize("dv", [-K.INF, K.INF])
def test_delta_limits(s, why, dv):
    """All gates open: the ordinary layer.  All gates shut: base path only, no conditional MMAs."""
    c = K.make_float_case("stlim", s, "bf16", delta=dv)
    ref, st, exempt, _ = _run(c, cond_mode=SKIP)
    assert exempt == 0
    if dv < 0:
        assert st.active == st.outputs and st.tiles_skipped == 0
    else:
        assert st.active == 0 and st.tiles_skipped == st.tiles_total > 0


@pytest.mark.parametrize("s,why", SHAPES[:4] + WIDE, ids=[w for _, w in SHAPES[:4] + WIDE])
def test_dense_mode_matches_skip_mode(s, why):
    c = K.make_float_case("stdense", s, "bf16", density=0.1, rho=0.7)
    ref, st_d, _, _ = _run(c, cond_mode=DENSE)
    _, st_s, _, _ = _run(c, cond_mode=SKIP)
    assert st_d.active == st_s.active
    assert st_d.tiles_skipped == 0
    assert st_s.executed_macs <= st_d.executed_macs


def test_idle_jobs_are_skipped():
    """Blank images give P = 0 below every (positive) threshold: their jobs issue no conditional
    MMAs, and the jobs around them still do."""
    s = O.Shape(8, 32, 32, 64, 64, groups=4)
    c = K.make_float_case("stskip", s, "bf16", density=0.05, rho=0.9)
    c.x[2:6] = 0.0
    t = O.fold_params(s, c.bn, c.delta)["t"]
    assert (t > 0).all()
    ref, st, _, plan = _run(c, cond_mode=SKIP)
    print(plan, st.tiles_skipped, st.tiles_total)
    assert st.tiles_skipped >= 4 * 8
    assert st.rows_active < st.rows_total


def test_ungated_layer_groups_1():
    """G = 1: the base path is the whole convolution (four K steps), there is no conditional path;
    the gate is still evaluated and selects between the two batch norms."""
    s = O.Shape(3, 32, 32, 64, 64, groups=1)
    c = K.make_float_case("stg1", s, "bf16", density=0.3)
    ref, st, exempt, _ = _run(c)
    assert st.gated_macs == st.dense_macs
    assert abs(st.density - ref.density) < 2e-3


def test_mask_pointer_may_be_null():
    s = O.Shape(3, 16, 16, 64, 64, groups=4)
    c = K.make_float_case("stnomask", s, "bf16", density=0.3)
    _run(c, with_mask=False)


def test_nan_input_does_not_fire():
    """A NaN partial sum compares false (gate shut) and the ReLU maps NaN to 0, as in the oracle;
    the pixels beside the 3x3 neighbourhood are untouched although their neighbours' stacked sums
    are NaN (image column 0 and W-1 drop, not multiply, what wraps around)."""
    s = O.Shape(2, 32, 32, 64, 64, groups=4)
    c = K.make_float_case("stnan", s, "bf16", density=0.3)
    c.x[0, 5, 0, 3] = np.nan          # a base-path channel in image column 0: outputs (4..6, 0..1) of image 0
    c.x[1, 7, 31, 2] = np.nan         # ... and in the last column
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=STACKED)
    y, mask, st = g.run()
    g.close()
    d_ref = O.unpack_mask(ref.mask, s.c_out)
    d_gpu = O.unpack_mask(mask, s.c_out)
    nan_rows = np.isnan(ref.p.reshape(-1, s.c_out)).any(axis=1)
    assert nan_rows.sum() == 12
    assert not d_gpu[nan_rows].any() and not d_ref[nan_rows].any()
    yr = y.reshape(-1, s.c_out)
    assert (yr[nan_rows] == 0).all() and (ref.y.reshape(-1, s.c_out)[nan_rows] == 0).all()
    ok = ~nan_rows
    assert not np.isnan(yr[ok]).any()
    np.testing.assert_array_equal(d_gpu[ok], d_ref[ok])


@pytest.mark.parametrize("s,why", [SHAPES[0], SHAPES[3], SHAPES[4]] + WIDE, ids=[w for _, w in [SHAPES[0], SHAPES[3], SHAPES[4]] + WIDE])
def test_residual_input(s, why):
    c = K.make_float_case("stres", s, "bf16", density=0.3, residual=True)
    ref, st, exempt, _ = _run(c)
    assert abs(st.density - ref.density) < 2e-3


@pytest.mark.parametrize("s", [O.Shape(3, 32, 32, 64, 64, groups=4), O.Shape(2, 56, 56, 64, 64, groups=4)], ids=["32x32", "56x56"])
def test_two_sided_gate(s):
    """Section 3.2: the gate fires only between the two thresholds."""
    c = K.make_float_case("st2s", s, "bf16", density=0.3)
    c.delta_high = (c.delta + np.float32(0.8)).astype(np.float32)
    ref, st, exempt, _ = _run(c)
    assert 0.02 < st.density < 0.28


def test_two_calls_accumulate_and_are_deterministic():
    s = O.Shape(2, 32, 32, 64, 64, groups=4)
    c = K.make_float_case("stdet", s, "bf16", density=0.3)
    g = K.GpuCase(c, algo=STACKED)
    y1, m1, st1 = g.run()
    y2, m2, st2 = g.run()
    np.testing.assert_array_equal(y1.view(np.uint32), y2.view(np.uint32))
    np.testing.assert_array_equal(m1, m2)
    assert st1.active == st2.active and st1.calls == st2.calls == 1
    g.close()


@pytest.mark.parametrize("workload,layer", [("cifar", "c64@32"), ("imagenet", "c64@56")])
def test_full_size_layer_on_sampled_images(workload, layer):
    """The 64-channel layers of the two benchmark workloads at benchmark batch; images are independent,
    so the oracle checks a sample of them one by one."""
    from paper_1805_12549_b200 import synth
    layers = synth.imagenet_resnet18_layers(64, 4) if workload == "imagenet" else synth.cifar_resnet18_layers(256, 4)
    ls = {l.name: l for l in layers}[layer]
    s = O.Shape(ls.n, ls.hw, ls.hw, ls.c_in, ls.c_out, stride=ls.stride, groups=4)
    c = K.make_float_case("stfull", s, "bf16", density=0.3, calib_images=2)
    g = K.GpuCase(c, algo=0 if workload == "cifar" else STACKED)   # (the default choice for the CIFAR layer)
    assert g.conv.kernel_id == 3, g.conv.plan
    y, mask, st = g.run()
    g.close()
    assert abs(st.density - 0.3) < 0.04
    per_img = s.ho * s.wo
    for n in sorted({0, s.n // 4 + 1, (5 * s.n) // 8, s.n - 1}):
        s1 = O.Shape(**{**s.__dict__, "n": 1})
        c1 = K.Case(c.name, s1, c.dtype, c.x[n:n + 1], c.wb, c.wc, c.bn, c.delta)
        ref = K.run_oracle(c1)
        K.compare(c1, ref, y[n:n + 1], mask[n * per_img:(n + 1) * per_img].reshape(-1, s.words), None)


def test_layers_outside_the_kernel_are_refused():
    from paper_1805_12549_b200 import binding as B
    for kw in (dict(w=130, h=8), dict(c_out=128), dict(groups=8), dict(k=1, pad=0), dict(stride=2)):
        a = dict(n=2, h=32, w=32, c_in=64, c_out=64, k=3, stride=1, pad=1, groups=4)
        a.update(kw)
        with pytest.raises(B.CgError):
            B.GatedConv(a["n"], a["h"], a["w"], a["c_in"], a["c_out"], k=a["k"], stride=a["stride"], pad=a["pad"],
                        groups=a["groups"], dtype=B.CG_BF16, algo=STACKED)
