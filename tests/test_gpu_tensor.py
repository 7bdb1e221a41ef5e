"""GPU parity of the pixel-major tcgen05 kernel (pixels on the MMA's M side) against the oracle.

bf16 bar: masks equal except where the oracle's normalised partial sum lies within 1e-3 of
Delta (that count is printed); outputs within 2e-2 + 1e-2*|ref| wherever the masks agree."""
import numpy as np
import pytest

from oracle import oracle as O
from tests import cases as K

pytestmark = pytest.mark.gpu

TENSOR = 3     # CG_ALGO_TENSOR_ROWS: this file pins the pixel-major kernel
DENSE, SKIP = 1, 2

# (shape, why): several tiles, ragged last tiles, every tiling mode
SHAPES = [
    (O.Shape(2, 56, 56, 64, 64, groups=4), "rows mode, 2 rows per tile, c_p = 16"),
    (O.Shape(3, 28, 28, 128, 128, groups=4), "rows mode, c_p = 32, two chunks"),
    (O.Shape(3, 14, 14, 256, 256, groups=4), "rows mode 7+7, c_p = 64, two column tiles"),
    (O.Shape(5, 7, 7, 512, 512, groups=4), "two images per tile, odd batch, c_p = 128"),
    (O.Shape(2, 32, 32, 64, 64, groups=4), "CIFAR 32x32"),
    (O.Shape(2, 16, 16, 128, 128, groups=4), "CIFAR 16x16"),
    (O.Shape(3, 8, 8, 256, 256, groups=4), "one 8x8 image per tile"),
    (O.Shape(7, 4, 4, 512, 512, groups=4), "five 4x4 images per tile, ragged"),
    (O.Shape(2, 28, 28, 128, 128, groups=8), "G = 8, c_p = 16"),
    (O.Shape(2, 14, 14, 256, 64, groups=8), "G = 8, c_p = 32, c_out != c_in"),
    (O.Shape(2, 13, 11, 64, 192, groups=2), "odd extents, G = 2, three column tiles of 64"),
    (O.Shape(2, 9, 9, 64, 64, kh=1, kw=1, pad=0, groups=4), "1x1 kernel"),
    (O.Shape(1, 5, 127, 64, 64, groups=4), "widest rows the kernel takes: 127 pixels + 1 pad column = one 128-row tile"),
    (O.Shape(1, 3, 3, 64, 64, groups=4), "one 3x3 image: a single, mostly empty tile"),
    (O.Shape(14, 56, 56, 64, 128, kh=1, kw=1, pad=0, groups=4), "1x1 kernel 64 -> 128, 392 row tiles: three jobs per CTA"),
    (O.Shape(12, 56, 56, 64, 64, groups=4), "336 row tiles: up to three jobs per CTA, resident weights"),
    (O.Shape(50, 28, 28, 128, 128, groups=4), "350 row tiles: streamed weights, three jobs per CTA"),
    (O.Shape(40, 14, 14, 256, 256, groups=4), "80 row tiles x 2 column tiles, two jobs per CTA"),
    (O.Shape(3, 56, 56, 64, 128, stride=2, groups=4), "stride 2, 56->28, c_p = 16"),
    (O.Shape(3, 28, 28, 128, 256, stride=2, groups=4), "stride 2, 28->14, c_p = 32"),
    (O.Shape(5, 14, 14, 256, 512, stride=2, groups=4), "stride 2, 14->7, c_p = 64, two images per tile"),
    (O.Shape(2, 12, 20, 64, 64, stride=2, groups=2), "stride 2, odd tile split, G = 2"),
    (O.Shape(3, 56, 56, 64, 64, groups=8), "G = 8 at 64 channels: c_p = 8 through repacked weights"),
    (O.Shape(3, 56, 56, 64, 128, stride=2, groups=8), "G = 8, stride 2, c_p = 8"),
    (O.Shape(2, 14, 14, 128, 64, groups=16), "G = 16 at 128 channels: c_p = 8, two chunks"),
]


def _run(c, cond_mode=0):
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=TENSOR, cond_mode=cond_mode)
    assert g.conv.uses_tensor_cores and g.conv.kernel_id == 1
    y, mask, st = g.run()
    exempt = K.compare(c, ref, y, mask, st)
    g.close()
    return ref, st, exempt


@pytest.mark.parametrize("s,why", SHAPES, ids=[w for _, w in SHAPES])
def test_parity_at_30_percent(s, why):
    c = K.make_float_case("tc30", s, "bf16", density=0.3)
    ref, st, exempt = _run(c)
    print(f"{why}: density {st.density:.3f}, near-tie mismatches {exempt}, "
          f"blocks skipped {st.tiles_skipped}/{st.tiles_total}")
    assert abs(st.density - ref.density) < 2e-3
    assert 0.2 < st.density < 0.4


@pytest.mark.parametrize("s,why", SHAPES[:4], ids=[w for _, w in SHAPES[:4]])
@pytest.mark.parametrize("dv", [-K.INF, K.INF])
def test_delta_limits(s, why, dv):
    """All gates open: the ordinary layer.  All gates shut: base path only, every block skipped."""
    c = K.make_float_case("tclim", s, "bf16", delta=dv)
    ref, st, exempt = _run(c)
    assert exempt == 0
    if dv < 0:
        assert st.active == st.outputs and st.tiles_skipped == 0
    else:
        assert st.active == 0 and st.tiles_skipped == st.tiles_total


@pytest.mark.parametrize("s,why", SHAPES[:4], ids=[w for _, w in SHAPES[:4]])
def test_dense_mode_matches_skip_mode(s, why):
    c = K.make_float_case("tcdense", s, "bf16", density=0.1, rho=0.7)
    ref, st_d, _ = _run(c, cond_mode=DENSE)
    _, st_s, _ = _run(c, cond_mode=SKIP)
    assert st_d.active == st_s.active
    assert st_d.tiles_skipped == 0
    assert st_s.executed_macs <= st_d.executed_macs


def test_idle_tiles_are_skipped():
    """A blank image gives P = 0 below every (positive) threshold: its tiles skip the
    conditional path entirely; clustered gates leave most pixel rows idle elsewhere."""
    s = O.Shape(2, 56, 56, 64, 64, groups=4)
    c = K.make_float_case("tcskip", s, "bf16", density=0.02, rho=0.95)
    c.x[1] = 0.0
    t = O.fold_params(s, c.bn, c.delta)["t"]
    assert (t > 0).all()
    ref, st, _ = _run(c, cond_mode=SKIP)
    assert st.tiles_total == 56 and st.tiles_skipped >= 28
    assert st.rows_active < st.rows_total // 2
    assert st.rows_total == s.m
    k2 = 9
    assert st.executed_macs == 128 * 64 * k2 * (s.c_p * 56 + s.c_r * (56 - st.tiles_skipped))


@pytest.mark.parametrize("dv", [K.INF, -K.INF])
def test_many_jobs_per_cta_all_shut_and_all_open(dv):
    """Several jobs per CTA with every conditional phase skipped (or none): the barrier phases
    of the skipped work must stay in step with the epilogue."""
    s = O.Shape(30, 28, 28, 128, 128, groups=4)          # 210 row tiles on 148 CTAs
    c = K.make_float_case("tcmany", s, "bf16", delta=dv)
    ref, st, exempt = _run(c)
    assert exempt == 0
    assert st.tiles_skipped == (st.tiles_total if dv > 0 else 0)


def test_two_calls_accumulate_and_are_deterministic():
    s = O.Shape(2, 28, 28, 128, 128, groups=4)
    c = K.make_float_case("tcdet", s, "bf16", density=0.3)
    g = K.GpuCase(c, algo=TENSOR)
    y1, m1, st1 = g.run()
    y2, m2, st2 = g.run()
    np.testing.assert_array_equal(y1.view(np.uint32), y2.view(np.uint32))
    np.testing.assert_array_equal(m1, m2)
    assert st1.active == st2.active and st1.calls == st2.calls == 1
    g.close()


@pytest.mark.parametrize("workload,layer", [
    ("imagenet", "c64@56"), ("imagenet", "c128@28"), ("imagenet", "c256@14"), ("imagenet", "c512@7"),
    ("imagenet", "c64to128@56s2"), ("imagenet", "c128to256@28s2"), ("imagenet", "c256to512@14s2"),
    ("cifar", "c64@32"), ("cifar", "c128@16"), ("cifar", "c256@8"), ("cifar", "c512@4")])
def test_full_size_layers_on_sampled_images(workload, layer):
    """Every layer shape of the two benchmark workloads (batch-64 ImageNet and batch-256 CIFAR
    ResNet-18 layers) in the configuration the benchmark times; images are independent, so the
    oracle checks a sample of them one by one."""
    from paper_1805_12549_b200 import synth
    layers = synth.imagenet_resnet18_layers(64, 4) if workload == "imagenet" else synth.cifar_resnet18_layers(256, 4)
    ls = {l.name: l for l in layers}[layer]
    s = O.Shape(ls.n, ls.hw, ls.hw, ls.c_in, ls.c_out, stride=ls.stride, groups=4)
    c = K.make_float_case("full", s, "bf16", density=0.3, calib_images=2)
    g = K.GpuCase(c, algo=TENSOR)
    assert g.conv.uses_tensor_cores
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


I8_SHAPES = [
    (O.Shape(2, 28, 28, 128, 128, groups=4), "int8 128@28, c_p = 32 bytes"),
    (O.Shape(3, 14, 14, 256, 256, groups=4), "int8 256@14, c_p = 64 bytes, two column tiles"),
    (O.Shape(5, 7, 7, 512, 512, groups=4), "int8 512@7, c_p = 128 bytes, two images per tile"),
    (O.Shape(2, 28, 28, 128, 256, stride=2, groups=4), "int8 stride 2"),
    (O.Shape(30, 28, 28, 128, 128, groups=2), "int8 G = 2, 210 row tiles"),
    (O.Shape(64, 28, 28, 128, 128, groups=4), "int8 128 -> 128, 448 row tiles: four jobs per CTA"),
    (O.Shape(3, 56, 56, 64, 64, groups=4), "int8 64@56: 64-byte pixel rows, half-empty column tile"),
    (O.Shape(2, 32, 32, 64, 64, groups=8), "int8 64@32, G = 8: 8 base channels"),
    (O.Shape(2, 56, 56, 64, 128, stride=2, groups=4), "int8 64 -> 128 stride 2"),
    (O.Shape(2, 28, 28, 128, 64, groups=4), "int8 128 -> 64: half-empty column tile"),
    (O.Shape(2, 14, 14, 256, 192, groups=4), "int8 256 -> 192: one full and one half-empty column tile"),
]


@pytest.mark.parametrize("s,why", I8_SHAPES, ids=[w for _, w in I8_SHAPES])
@pytest.mark.parametrize("density", [0.3, 1.0, 0.0])
def test_int8_tensor_path_is_bit_exact(s, why, density):
    """Quantised layers on tcgen05 kind::i8: integer sums are order-independent, so masks and
    int8 outputs must equal the oracle's bit for bit."""
    c = K.make_int8_case("tci8", s, density=density)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=TENSOR)
    assert g.conv.uses_tensor_cores
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st, exact=True)
    assert st.active == ref.active
    if density == 0.3:
        assert 0.2 < st.density < 0.4 and len(np.unique(y)) > 16
    g.close()


COMPACT = 3
COMPACT_CASES = [
    (O.Shape(2, 56, 56, 64, 64, groups=4), 0.3, 0.0, "c_p = 16, every row active"),
    (O.Shape(3, 28, 28, 128, 128, groups=4), 0.05, 0.9, "c_p = 32, clustered gates"),
    (O.Shape(3, 14, 14, 256, 256, groups=4), 0.1, 0.8, "c_p = 64, two column tiles"),
    (O.Shape(5, 7, 7, 512, 512, groups=4), 0.02, 0.95, "c_p = 128, few rows"),
    (O.Shape(3, 28, 28, 128, 256, stride=2, groups=4), 0.1, 0.5, "stride 2"),
    (O.Shape(20, 28, 28, 128, 128, groups=8), 0.3, 0.0, "G = 8, many row groups per CTA"),
]


@pytest.mark.parametrize("s,density,rho,why", COMPACT_CASES, ids=[c[3] for c in COMPACT_CASES])
def test_row_compaction_mode(s, density, rho, why):
    """CG_COND_COMPACT: the first kernel lists the pixel rows with a firing gate, the second
    gathers those rows into dense sub-GEMMs for the conditional path (Eq. 1, second case)."""
    c = K.make_float_case("tccomp", s, "bf16", density=density, rho=rho)
    ref = K.run_oracle(c)
    g = K.GpuCase(c, algo=TENSOR, cond_mode=COMPACT)
    assert g.conv.workspace is not None
    y, mask, st = g.run()
    K.compare(c, ref, y, mask, st)
    assert st.rows_total % s.m == 0          # pixel rows x column tiles
    print(f"{why}: density {st.density:.3f}, rows active {st.rows_active}/{st.rows_total}, "
          f"executed/gated MACs {st.executed_macs / st.gated_macs:.2f}")
    # a second call reuses the workspace
    y2, mask2, _ = g.run()
    np.testing.assert_array_equal(y.view(np.uint32), y2.view(np.uint32))
    g.close()


def test_compaction_with_no_active_rows_and_all_rows():
    s = O.Shape(2, 28, 28, 128, 128, groups=4)
    for dv in (K.INF, -K.INF):
        c = K.make_float_case("tccomp2", s, "bf16", delta=dv)
        ref = K.run_oracle(c)
        g = K.GpuCase(c, algo=TENSOR, cond_mode=COMPACT)
        y, mask, st = g.run()
        K.compare(c, ref, y, mask, st)
        g.close()


RESIDUAL_SHAPES = [
    (O.Shape(3, 28, 28, 128, 128, groups=4), "streamed weights, NT = 128"),
    (O.Shape(2, 56, 56, 64, 64, groups=4), "resident weights, two issuers"),
    (O.Shape(7, 4, 4, 512, 512, groups=4), "images per tile, ragged batch"),
    (O.Shape(3, 28, 28, 128, 256, stride=2, groups=4), "stride 2"),
]


@pytest.mark.parametrize("s,why", RESIDUAL_SHAPES, ids=[w for _, w in RESIDUAL_SHAPES])
def test_residual_input_on_the_tensor_path(s, why):
    """The shortcut of a residual block is added after the batch norm and before the ReLU
    (second convolution of a block, Fig. 2 / Section 4)."""
    c = K.make_float_case("tcres", s, "bf16", density=0.3, residual=True)
    ref, st, exempt = _run(c)
    assert abs(st.density - ref.density) < 2e-3
    # the residual changes the output: without it the result must differ
    c0 = K.make_float_case("tcres", s, "bf16", density=0.3, residual=False)
    ref0 = K.run_oracle(c0)
    assert np.abs(ref.y.astype(np.float64) - ref0.y.astype(np.float64)).max() > 0.1


def test_dependent_layers_back_to_back_on_one_stream():
    """Two layers chained on one stream without any host synchronisation: the second reads the
    first one's output.  Each call is a programmatic dependent launch (its blocks may start while
    the previous kernel drains), so this checks that no block touches global memory before the
    previous kernel has finished: the result must be bit-identical to the same chain run with a
    device synchronisation after every call, on every one of several repetitions."""
    import torch
    s = O.Shape(24, 28, 28, 128, 128, groups=4)
    c = K.make_float_case("chain", s, "bf16", density=0.3, calib_images=2)
    g1 = K.GpuCase(c, algo=TENSOR)
    g2 = K.GpuCase(c, algo=TENSOR)
    assert g1.conv.uses_tensor_cores

    def chain(sync):
        g1.y.fill_(0); g2.y.fill_(0); g2.mask.fill_(-1)
        torch.cuda.synchronize()
        for _ in range(3):     # the last pass decides; earlier passes keep the queue full
            g1.conv.forward(g1.x, g1.wb, g1.wc, g1.bn, g1.delta, g1.y, g1.mask, None)
            if sync:
                torch.cuda.synchronize()
            g2.conv.forward(g1.y, g2.wb, g2.wc, g2.bn, g2.delta, g2.y, g2.mask, None)
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        return g2.y.clone(), g2.mask.clone()

    y_ref, m_ref = chain(sync=True)
    for _ in range(5):
        y, m = chain(sync=False)
        assert torch.equal(m, m_ref)
        assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16))
    assert g1.conv.stats().device_status == 0 and g2.conv.stats().device_status == 0
    g1.close(); g2.close()


def test_misaligned_workspace_is_refused_before_any_launch():
    """cg_conv_forward checks the workspace pointer (256-byte alignment) on the host."""
    import torch
    from paper_1805_12549_b200 import binding as B
    s = O.Shape(2, 28, 28, 128, 128, groups=4)
    c = K.make_float_case("tcalign", s, "bf16", density=0.3)
    g = K.GpuCase(c, algo=TENSOR, cond_mode=3)               # row compaction: the layer needs a workspace
    need = B.cg_conv_workspace_bytes(g.conv.handle)
    assert need > 0
    y0, m0, _ = g.run()
    buf = torch.zeros(need + 512, dtype=torch.uint8, device="cuda")
    off = (-buf.data_ptr()) % 256 + 16
    g.conv.workspace = buf[off:off + need]
    g.y.fill_(0)
    with pytest.raises(B.CgError) as e:
        g.conv.forward(g.x, g.wb, g.wc, g.bn, g.delta, g.y, g.mask, g.res)
    assert e.value.status == 3                               # CG_ERR_ALIGNMENT
    torch.cuda.synchronize()
    assert float(g.y.float().abs().max()) == 0.0             # nothing ran
    g.conv.workspace = None
    with pytest.raises(B.CgError) as e:
        g.conv.forward(g.x, g.wb, g.wc, g.bn, g.delta, g.y, g.mask, g.res)
    assert e.value.status == 4                               # CG_ERR_WORKSPACE
    g.close()


GROUPED = [
    (O.Shape(3, 14, 14, 256, 256, groups=4), "256 channels, G = 4: column tiles of 64 inside the groups"),
    (O.Shape(5, 7, 7, 512, 512, groups=4), "512 channels, G = 4: column tiles of 128"),
    (O.Shape(2, 14, 14, 256, 512, groups=4), "c_out != c_in"),
    (O.Shape(2, 28, 28, 128, 128, groups=2), "G = 2 at 128 channels"),
    (O.Shape(3, 14, 14, 256, 512, stride=2, groups=4), "stride 2"),
    (O.Shape(2, 14, 14, 512, 512, groups=8), "G = 8 at 512 channels: groups of 64"),
]


@pytest.mark.parametrize("s,why", GROUPED, ids=[w for _, w in GROUPED])
def test_channel_grouping_on_the_tensor_path(s, why):
    """Section 3.3: output group i takes input group i as its base path and the other groups, in
    ascending order, as its conditional path."""
    c = K.make_float_case("tcgrp", s, "bf16", density=0.3, grouped=True)
    ref, st, exempt = _run(c)
    assert abs(st.density - ref.density) < 2e-3 and 0.2 < st.density < 0.4
    c = K.make_float_case("tcgrp1", s, "bf16", delta=-K.INF, grouped=True)
    ref, st, exempt = _run(c)
    assert exempt == 0 and st.active == st.outputs


CHANNEL_GATE = [
    (O.Shape(3, 28, 28, 128, 128, groups=4), "128@28"),
    (O.Shape(3, 14, 14, 256, 256, groups=4), "256@14, two column tiles"),
    (O.Shape(2, 56, 56, 64, 64, groups=4), "64@56, one patch for both paths"),
    (O.Shape(3, 28, 28, 128, 256, stride=2, groups=4), "stride 2"),
    (O.Shape(5, 7, 7, 512, 512, groups=4), "two images per tile: thresholds per image inside a tile"),
]


@pytest.mark.parametrize("s,why", CHANNEL_GATE, ids=[w for _, w in CHANNEL_GATE])
@pytest.mark.parametrize("tau", [0.3, 0.45])
def test_channel_wise_gate_on_the_tensor_path(s, why, tau):
    """Eq. 4 as two passes of the pixel-major kernel: the first counts the plain gate's decisions per
    (image, channel), the second runs the layer with the switched-off channels' thresholds at +inf."""
    c = K.make_float_case("tcchan", s, "bf16", density=0.4)
    c.channel_tau = tau
    ref, st, exempt = _run(c)
    assert st.channels == ref.channels == s.n * s.c_out
    assert st.channels_skipped == ref.channels_skipped
    assert st.channels_skipped < st.channels
    if tau > 0.4:
        assert st.channels_skipped > 0, "the case should drop some channels"
    assert st.calls == 1 and st.device_status == 0


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
    ref, st, exempt = _run(c)
    assert 0 < ref.active < one_sided.active
    assert st.active == ref.active or exempt > 0
