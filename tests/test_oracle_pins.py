"""Pins for the CPU oracle: each test checks it against something other than itself --
a library convolution, a closed form, a hand-computed case, exact integer arithmetic.

Citations are to Channel Gating Neural Networks (arXiv 1805.12549).
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import oracle as O
from paper_1805_12549_b200 import synth

INF = float("inf")


# ----------------------------------------------------------------------------- helpers
def make_layer(key, s: O.Shape, separate=True, smooth=False):
    if smooth:
        x = synth.smoothed_noise((key, "x"), s.n, s.h, s.w, s.c_in)
    else:
        x = synth.rng(key, "x").standard_normal((s.n, s.h, s.w, s.c_in), dtype=np.float32)
    wb, wc = synth.kaiming_weights(key, s.c_out, s.kh, s.kw, s.c_in, s.groups)
    bn = synth.bn_params(key, s.c_out, separate=separate)
    return x, wb, wc, bn


def lib_conv64(x, w, stride, pad, groups=1):
    """Library convolution in fp64.  x [N,H,W,C], w [Co,kh,kw,Ci] -> [N,H',W',Co]."""
    xt = torch.from_numpy(np.asarray(x, np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(np.asarray(w, np.float64)).permute(0, 3, 1, 2)
    return F.conv2d(xt, wt, stride=stride, padding=pad, groups=groups).permute(0, 2, 3, 1).numpy()


def bn_relu64(v, gamma, beta, mean, var, eps, relu=True):
    out = gamma.astype(np.float64) * (v - mean.astype(np.float64)) / np.sqrt(
        var.astype(np.float64) + eps) + beta.astype(np.float64)
    return np.maximum(out, 0.0) if relu else out


SHAPES = [
    O.Shape(2, 8, 8, 16, 16, groups=4),
    O.Shape(1, 7, 9, 8, 5, groups=2),
    O.Shape(2, 9, 9, 12, 7, stride=2, groups=4),
    O.Shape(1, 6, 6, 6, 4, kh=1, kw=1, pad=0, groups=3),
    O.Shape(1, 8, 8, 4, 3, kh=5, kw=5, pad=2, groups=2),
    O.Shape(1, 8, 7, 8, 6, stride=2, pad=0, groups=8),
]


# ----------------------------------------------------------------------------- T1 / T2
@pytest.mark.parametrize("s", SHAPES)
def test_open_gate_is_dense_conv(s):
    """Section 3.1: W*x = W_p*x_p + W_r*x_r, so with every gate open (Delta=-inf) Eq. 1's
    second case gives the ordinary layer f(BN2(W*x))."""
    x, wb, wc, bn = make_layer(("t1", s.c_in, s.h), s)
    res = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, -INF, np.float32))
    w_full = np.concatenate([wb, wc], axis=3)
    ref = bn_relu64(lib_conv64(x, w_full, s.stride, s.pad), bn["gamma"], bn["beta"],
                    bn["mean_full"], bn["var_full"], s.bn_eps)
    np.testing.assert_allclose(res.y, ref, rtol=1e-5, atol=1e-5)
    assert res.active == res.outputs == s.m * s.c_out
    assert O.unpack_mask(res.mask, s.c_out).all()
    # unused high bits of the last mask word stay zero
    if s.c_out % 32:
        assert (res.mask[:, -1] >> (s.c_out % 32)).max() == 0


@pytest.mark.parametrize("s", SHAPES)
def test_shut_gate_is_base_path_only(s):
    """Eq. 1, first case: with every gate shut (Delta=+inf) y = f(BN1(W_p*x_p))."""
    x, wb, wc, bn = make_layer(("t2", s.c_in, s.h), s)
    res = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, INF, np.float32))
    p_ref = lib_conv64(x[..., :s.c_p], wb, s.stride, s.pad)
    ref = bn_relu64(p_ref, bn["gamma"], bn["beta"], bn["mean_base"], bn["var_base"], s.bn_eps)
    np.testing.assert_allclose(res.y, ref, rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(res.p, p_ref, rtol=1e-5, atol=1e-5)
    assert res.active == 0 and res.cond_macs == 0
    assert not res.mask.any()


@pytest.mark.parametrize("s", SHAPES[:3])
def test_mixed_gate_selects_per_activation(s):
    """Eq. 1 at a finite Delta: every activation equals one of the two library results, chosen
    by the library partial sum against Eq. 3's threshold (away from near-ties)."""
    x, wb, wc, bn = make_layer(("mix", s.c_in, s.h), s)
    delta = synth.rng("mix-delta", s.c_in).uniform(-0.5, 0.5, s.c_out).astype(np.float32)
    res = O.gated_conv(s, x, wb, wc, bn, delta)
    p_ref = lib_conv64(x[..., :s.c_p], wb, s.stride, s.pad)
    full_ref = lib_conv64(x, np.concatenate([wb, wc], axis=3), s.stride, s.pad)
    t = delta.astype(np.float64) * np.sqrt(bn["gate_var"].astype(np.float64) + s.bn_eps) \
        + bn["gate_mean"].astype(np.float64)
    d_ref = p_ref >= t
    clear = np.abs(p_ref - t) > 1e-4
    d = O.unpack_mask(res.mask, s.c_out).reshape(p_ref.shape)
    assert (d == d_ref)[clear].all()
    y_ref = np.where(d, bn_relu64(full_ref, bn["gamma"], bn["beta"], bn["mean_full"],
                                  bn["var_full"], s.bn_eps),
                     bn_relu64(p_ref, bn["gamma"], bn["beta"], bn["mean_base"], bn["var_base"],
                               s.bn_eps))
    np.testing.assert_allclose(res.y, y_ref, rtol=1e-5, atol=1e-5)
    assert 0 < res.active < res.outputs
    assert res.active == int(d.sum())


def test_residual_is_added_before_relu():
    s = O.Shape(1, 6, 6, 8, 8, groups=4)
    x, wb, wc, bn = make_layer("res", s)
    r = synth.residual("res", (s.n, s.ho, s.wo, s.c_out))
    delta = np.zeros(s.c_out, np.float32)
    plain = O.Shape(**{**s.__dict__, "relu": 0})
    pre = O.gated_conv(plain, x, wb, wc, bn, delta)
    got = O.gated_conv(s, x, wb, wc, bn, delta, residual=r)
    np.testing.assert_allclose(got.y, np.maximum(pre.y.astype(np.float64) + r, 0), rtol=1e-6,
                               atol=1e-6)
    assert (got.mask == pre.mask).all()


# ----------------------------------------------------------------------------- hand case, T3
def _read_golden(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = np.array([float(t) for t in v])
    return out


def test_hand_case(golden_dir):
    """The 3x3 case of tests/golden/hand_case.txt, worked by hand from Eq. 1-3; includes an
    exact tie that must fire (Eq. 2: theta(0) = 1)."""
    g = _read_golden(os.path.join(golden_dir, "hand_case.txt"))
    s = O.Shape(1, 3, 3, 2, 1, groups=2, bn_eps=0.0)
    x = np.stack([g["x_p"].reshape(3, 3), g["x_r"].reshape(3, 3)], axis=-1)[None]
    wb = np.ones((1, 3, 3, 1), np.float32)
    wc = np.zeros((1, 3, 3, 1), np.float32)
    wc[0, 1, 1, 0] = 1.0
    bn = {k: g[k].astype(np.float32) for k in ("gamma", "beta", "mean_base", "var_base",
                                               "mean_full", "var_full", "gate_mean", "gate_var")}
    res = O.gated_conv(s, x, wb, wc, bn, g["delta"].astype(np.float32))
    np.testing.assert_array_equal(res.p.reshape(-1), g["P"])
    np.testing.assert_array_equal(O.unpack_mask(res.mask, 1).reshape(-1), g["d"].astype(bool))
    np.testing.assert_allclose(res.y.reshape(-1), g["y"], rtol=0, atol=2e-6)
    assert res.base_macs == int(g["base_macs"][0])
    assert res.cond_macs == int(g["cond_macs"][0])
    assert res.dense_macs == int(g["dense_macs"][0])
    assert res.active == 5
    # reduction 162/126 = 1/(eta + (1-eta)*tau), eta = 1/2, tau = 5/9
    assert math.isclose(res.dense_macs / res.gated_macs, 1.0 / (0.5 + 0.5 * 5 / 9), rel_tol=1e-12)


def test_tie_fires_and_just_below_does_not():
    """Eq. 2: x >= 0 gives 1.  One channel, 1x1 kernel, so P = x exactly."""
    s = O.Shape(1, 1, 4, 2, 1, kh=1, kw=1, pad=0, groups=2, bn_eps=0.0)
    x = np.zeros((1, 1, 4, 2), np.float32)
    x[0, 0, :, 0] = [3.0, np.nextafter(np.float32(3.0), np.float32(0.0)), 3.5, np.nan]
    x[0, 0, :, 1] = 1.0
    wb = np.ones((1, 1, 1, 1), np.float32)
    wc = np.ones((1, 1, 1, 1), np.float32)
    one, zero = np.ones(1, np.float32), np.zeros(1, np.float32)
    bn = dict(gamma=one, beta=zero, mean_base=zero, var_base=one, mean_full=zero, var_full=one,
              gate_mean=one, gate_var=np.full(1, 4.0, np.float32))
    res = O.gated_conv(s, x, wb, wc, bn, np.ones(1, np.float32))     # t = 1*2 + 1 = 3
    assert O.unpack_mask(res.mask, 1).reshape(-1).tolist() == [True, False, True, False]
    assert res.y.reshape(-1)[:3].tolist() == [4.0, float(x[0, 0, 1, 0]), 4.5]
    assert res.y.reshape(-1)[3] == 0.0                               # NaN: gate shut, ReLU -> 0


# ----------------------------------------------------------------------------- T4, T5, T6
def test_merged_gate_equals_normalise_then_compare():
    """Section 3.2: normalising P with (E, Var) and comparing with Delta is the same decision
    as Eq. 3's merged threshold, because sqrt(Var) > 0."""
    s = O.Shape(2, 10, 10, 16, 24, groups=4)
    x, wb, wc, bn = make_layer("t4", s)
    delta = synth.rng("t4-delta").uniform(-1, 1, s.c_out).astype(np.float32)
    a = O.gated_conv(s, x, wb, wc, bn, delta, gate_form=0)
    b = O.gated_conv(s, x, wb, wc, bn, delta, gate_form=1)
    da, db = O.unpack_mask(a.mask, s.c_out), O.unpack_mask(b.mask, s.c_out)
    p_hat = (a.p.reshape(-1, s.c_out) - bn["gate_mean"]) / np.sqrt(bn["gate_var"] + s.bn_eps)
    clear = np.abs(p_hat - delta) > 1e-5
    assert (da == db)[clear].all()
    assert (da != db).sum() <= (~clear).sum()


def test_mask_shrinks_as_delta_grows():
    """Section 4, "Inducing sparsity": the pruned fraction rises monotonically with Delta."""
    s = O.Shape(2, 12, 12, 16, 16, groups=4)
    x, wb, wc, bn = make_layer("t5", s, smooth=True)
    prev = None
    for dv in (-2.0, -0.5, 0.0, 0.5, 2.0):
        m = O.unpack_mask(O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, dv, np.float32)).mask,
                          s.c_out)
        if prev is not None:
            assert not (m & ~prev).any()
            assert m.sum() < prev.sum()
        prev = m


@pytest.mark.parametrize("dv", [-1.0, 0.0, 1.0, 1.5, 2.0])
def test_firing_rate_matches_normal_tail(dv):
    """Section 4: the normalised gate input is standard normal, so the firing rate is
    1 - Phi(Delta).  With iid N(0,1) inputs and no padding, P[.,c] is exactly N(0, |W_p[c]|^2);
    those closed-form statistics are handed to the gate."""
    s = O.Shape(4, 34, 34, 8, 8, pad=0, groups=2, bn_eps=0.0)
    x, wb, wc, bn = make_layer("t6", s)
    bn = dict(bn)
    bn["gate_mean"] = np.zeros(s.c_out, np.float32)
    bn["gate_var"] = (wb.astype(np.float64) ** 2).sum(axis=(1, 2, 3)).astype(np.float32)
    res = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, dv, np.float32))
    expect = 0.5 * math.erfc(dv / math.sqrt(2.0))
    # neighbouring outputs share inputs: allow 6 sigma of an effective sample 1/9 the size
    tol = 6.0 * math.sqrt(expect * (1 - expect) / (res.outputs / 9.0))
    assert abs(res.density - expect) < tol


# ----------------------------------------------------------------------------- T7
@pytest.mark.parametrize("s", SHAPES)
def test_multiplication_count_closed_form(s):
    """Section 4: base path costs eta*c_l*k^2 multiplications per output activation, the
    conditional path (1-eta)*c_l*k^2 per firing activation; padding taps are counted."""
    x, wb, wc, bn = make_layer(("t7", s.c_in), s)
    res = O.gated_conv(s, x, wb, wc, bn, np.zeros(s.c_out, np.float32))
    n_out = s.n * s.ho * s.wo * s.c_out
    k2 = s.kh * s.kw
    assert res.outputs == n_out
    assert res.base_macs == k2 * s.c_p * n_out
    assert res.cond_macs == k2 * s.c_r * res.active
    assert res.dense_macs == k2 * s.c_in * n_out
    eta, tau = 1.0 / s.groups, res.active / n_out
    assert math.isclose(res.dense_macs / res.gated_macs, 1.0 / (eta + (1 - eta) * tau),
                        rel_tol=1e-12)
    assert res.active == int(O.unpack_mask(res.mask, s.c_out).sum())


# ----------------------------------------------------------------------------- precision variants
def test_double_accumulation_envelope_and_bf16_rounding():
    s = O.Shape(2, 8, 8, 32, 32, groups=4)
    x, wb, wc, bn = make_layer("acc", s, smooth=True)
    x, wb, wc = synth.bf16_round(x), synth.bf16_round(wb), synth.bf16_round(wc)
    delta = np.zeros(s.c_out, np.float32)
    a = O.gated_conv(s, x, wb, wc, bn, delta)
    b = O.gated_conv(s, x, wb, wc, bn, delta, acc_double=True)
    assert np.abs(a.p - b.p).max() < 1e-5
    same = O.unpack_mask(a.mask, s.c_out) == O.unpack_mask(b.mask, s.c_out)
    assert same.mean() > 0.999
    c = O.gated_conv(s, x, wb, wc, bn, delta, out_bf16=True)
    # bf16 output is the fp32 output rounded to 8 significant bits, nearest even
    np.testing.assert_array_equal(c.y, synth.bf16_round(a.y))
    ref = torch.from_numpy(a.y).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(c.y, ref)


def test_fold_params_matches_fp64_within_half_ulp():
    s = O.Shape(1, 4, 4, 8, 64, groups=4)
    bn = synth.bn_params("fold", s.c_out)
    delta = synth.rng("fold-d").uniform(-2, 2, s.c_out).astype(np.float32)
    f = O.fold_params(s, bn, delta)
    t64 = delta.astype(np.float64) * np.sqrt(bn["gate_var"].astype(np.float64) + s.bn_eps) \
        + bn["gate_mean"]
    a64 = bn["gamma"] / np.sqrt(bn["var_full"].astype(np.float64) + s.bn_eps)
    np.testing.assert_allclose(f["t"], t64, rtol=3e-7, atol=1e-7)
    np.testing.assert_allclose(f["a2"], a64, rtol=3e-7)
    np.testing.assert_allclose(f["b2"], bn["beta"] - a64 * bn["mean_full"], rtol=1e-6, atol=1e-7)
    # gate statistics default to BN1's (both normalise the partial sum)
    bn2 = {k: v for k, v in bn.items() if not k.startswith("gate_")}
    f2 = O.fold_params(s, bn2, delta)
    t1 = delta.astype(np.float64) * np.sqrt(bn["var_base"].astype(np.float64) + s.bn_eps) \
        + bn["mean_base"]
    np.testing.assert_allclose(f2["t"], t1, rtol=3e-7, atol=1e-7)


# ----------------------------------------------------------------------------- config 1
@pytest.mark.parametrize("separate", [False, True])
def test_config1_density_is_about_half(separate):
    s = O.Shape(2, 8, 8, 16, 16, groups=4)
    x, wb, wc, bn = make_layer(("cfg1", separate), s, separate=separate)
    res = O.gated_conv(s, x, wb, wc, bn, np.zeros(s.c_out, np.float32))
    assert 0.3 < res.density < 0.7
    assert res.y.shape == (2, 8, 8, 16) and (res.y >= 0).all()


# ----------------------------------------------------------------------------- channel grouping
def test_grouped_base_path_is_a_grouped_convolution():
    """Section 3.3: with channel grouping the base path is an ordinary grouped convolution, and
    output group i takes the other input groups, in order, as x_r."""
    s = O.Shape(2, 7, 7, 12, 8, groups=4)
    x, wb, wc, bn = make_layer("grp", s)
    shut = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, INF, np.float32), grouped=True)
    p_ref = lib_conv64(x, wb, s.stride, s.pad, groups=s.groups)
    np.testing.assert_allclose(shut.p, p_ref, rtol=1e-5, atol=1e-5)
    # all-open: reassemble a dense weight tensor and compare with a dense convolution
    cp, og = s.c_p, s.c_out // s.groups
    w_full = np.zeros((s.c_out, 3, 3, s.c_in), np.float32)
    for co in range(s.c_out):
        g = co // og
        w_full[co, :, :, g * cp:(g + 1) * cp] = wb[co]
        others = [c for c in range(s.c_in) if c // cp != g]
        w_full[co][:, :, others] = wc[co]
    opened = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, -INF, np.float32), grouped=True)
    ref = bn_relu64(lib_conv64(x, w_full, s.stride, s.pad), bn["gamma"], bn["beta"],
                    bn["mean_full"], bn["var_full"], s.bn_eps)
    np.testing.assert_allclose(opened.y, ref, rtol=1e-5, atol=1e-5)


# ----------------------------------------------------------------------------- int8
def _py_requant(acc, mul, off, shift, relu):
    z = int(acc) * int(mul) + int(off)          # Python integers: exact
    q = (z + (1 << (shift - 1))) >> shift       # floor division by 2^S: arithmetic shift
    return max(0 if relu else -128, min(127, q))


@pytest.mark.parametrize("s,shift", [(O.Shape(1, 5, 5, 8, 6, groups=4), 24),
                                     (O.Shape(2, 6, 5, 16, 9, stride=2, groups=2), 16),
                                     (O.Shape(1, 4, 4, 4, 3, groups=4, relu=0), 20)])
def test_int8_layer_exact(s, shift):
    x = synth.int8_activations(("i8", s.c_in), s.n, s.h, s.w, s.c_in)
    wb, wc = synth.int8_weights(("i8", s.c_in), s.c_out, s.kh, s.kw, s.c_in, s.groups)
    # integer convolutions by the library routine (exact in int64)
    xt = torch.from_numpy(x.astype(np.int64)).permute(0, 3, 1, 2)
    conv = lambda xx, ww: F.conv2d(xx, torch.from_numpy(ww.astype(np.int64)).permute(0, 3, 1, 2),
                                   stride=s.stride, padding=s.pad).permute(0, 2, 3, 1).numpy()
    p_ref = conv(xt[:, :s.c_p], wb)
    r_ref = conv(xt[:, s.c_p:], wc)
    q = synth.int8_requant(("i8", s.c_in), s.c_out, shift, p_ref.std() + 1, (p_ref + r_ref).std() + 1)
    q["q_gate_thr"] = np.median(p_ref.reshape(-1, s.c_out), axis=0).astype(np.int32)
    if not s.relu:
        q["q_off_base"] = q["q_off_base"] - (40 << shift)   # reach the negative clamp too
    res = O.gated_conv_i8(s, shift, x, wb, wc, q)
    np.testing.assert_array_equal(res.p, p_ref)
    d_ref = p_ref >= q["q_gate_thr"][None, None, None, :]
    np.testing.assert_array_equal(O.unpack_mask(res.mask, s.c_out).reshape(d_ref.shape), d_ref)
    y_ref = np.empty(p_ref.shape, np.int64)
    for idx in np.ndindex(*p_ref.shape):
        c = idx[-1]
        if d_ref[idx]:
            y_ref[idx] = _py_requant(p_ref[idx] + r_ref[idx], q["q_mul_full"][c], q["q_off_full"][c],
                                     shift, s.relu)
        else:
            y_ref[idx] = _py_requant(p_ref[idx], q["q_mul_base"][c], q["q_off_base"][c], shift,
                                     s.relu)
    np.testing.assert_array_equal(res.y.astype(np.int64), y_ref)
    assert len(np.unique(res.y)) > 8            # not collapsed onto a clamp
    assert res.cond_macs == s.kh * s.kw * s.c_r * int(d_ref.sum())


def test_int8_threshold_limits():
    s = O.Shape(1, 5, 5, 8, 4, groups=4)
    x = synth.int8_activations("i8lim", s.n, s.h, s.w, s.c_in)
    wb, wc = synth.int8_weights("i8lim", s.c_out, 3, 3, s.c_in, s.groups)
    q = synth.int8_requant("i8lim", s.c_out, 20, 500.0, 1500.0)
    q["q_gate_thr"] = np.full(s.c_out, np.iinfo(np.int32).min, np.int32)
    assert O.gated_conv_i8(s, 20, x, wb, wc, q).active == s.m * s.c_out
    q["q_gate_thr"] = np.full(s.c_out, np.iinfo(np.int32).max, np.int32)
    assert O.gated_conv_i8(s, 20, x, wb, wc, q).active == 0


# ----------------------------------------------------------------------------- channel-wise gate
def _golden(name):
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            out[k] = np.array([float(t) for t in v])
    return out


def test_channel_gate_hand_case():
    """Eq. 4 on the worked example of tests/golden/channel_gate_case.txt (per-image counts,
    ties keep the channel, a dropped channel takes Eq. 1's first case everywhere)."""
    g = _golden("channel_gate_case.txt")
    s = O.Shape(2, 2, 2, 2, 2, kh=1, kw=1, pad=0, groups=2, bn_eps=0.0)
    x = np.stack([g["x_p"], g["x_r"]], axis=-1).reshape(2, 2, 2, 2).astype(np.float32)
    wb = np.array([1.0, 2.0], np.float32).reshape(2, 1, 1, 1)
    wc = np.array([1.0, -1.0], np.float32).reshape(2, 1, 1, 1)
    one, zero = np.ones(2, np.float32), np.zeros(2, np.float32)
    bn = dict(gamma=one, beta=zero, mean_base=zero, var_base=one, mean_full=zero, var_full=one,
              gate_mean=zero, gate_var=one)
    for tag in ("a", "b"):
        res = O.gated_conv(s, x, wb, wc, bn, g["delta"].astype(np.float32),
                           channel_tau=float(g["tau_" + tag][0]))
        d = O.unpack_mask(res.mask, 2).reshape(-1).astype(int)
        assert d.tolist() == g["d_" + tag].astype(int).tolist()
        np.testing.assert_array_equal(res.y.reshape(-1), g["y_" + tag].astype(np.float32))
        assert res.channels == 4 and res.channels_skipped == int(g["skipped_" + tag][0])
        assert res.cond_macs == int(g["cond_macs_" + tag][0]) and res.active == res.cond_macs


@pytest.mark.parametrize("s", SHAPES[:3])
def test_channel_gate_limits(s):
    """Eq. 4: tau_c = 0 keeps every channel (any count >= 0), so the layer is unchanged;
    tau_c > 1 drops every channel (no count reaches more than w*h), so the layer is the base
    path alone, as with Delta = +inf."""
    x, wb, wc, bn = make_layer(("cg-lim", s.c_in, s.h), s)
    delta = np.zeros(s.c_out, np.float32)
    plain = O.gated_conv(s, x, wb, wc, bn, delta)
    off = O.gated_conv(s, x, wb, wc, bn, delta, channel_tau=0.0)
    np.testing.assert_array_equal(plain.y, off.y)
    np.testing.assert_array_equal(plain.mask, off.mask)
    assert off.channels_skipped == 0
    shut = O.gated_conv(s, x, wb, wc, bn, delta, channel_tau=1.5)
    base = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, INF, np.float32))
    np.testing.assert_array_equal(shut.y, base.y)
    assert not shut.mask.any() and shut.active == 0
    assert shut.channels_skipped == shut.channels == s.n * s.c_out


@pytest.mark.parametrize("s", SHAPES[:3])
@pytest.mark.parametrize("tau", [0.35, 0.45, 0.55])
def test_channel_gate_restated_with_numpy(s, tau):
    """Eq. 4 restated on the activation-wise decisions: per image and channel, count the firing
    gates over the feature map, keep the channel iff count >= tau_c*w*h, and AND that with the
    activation-wise mask; the conditional path runs exactly on the surviving activations."""
    x, wb, wc, bn = make_layer(("cg-np", s.c_in, s.h), s)
    delta = synth.rng("cg-np-delta", s.c_in).uniform(-0.3, 0.3, s.c_out).astype(np.float32)
    plain = O.gated_conv(s, x, wb, wc, bn, delta)
    res = O.gated_conv(s, x, wb, wc, bn, delta, channel_tau=tau)
    d = O.unpack_mask(plain.mask, s.c_out).reshape(s.n, s.ho * s.wo, s.c_out)
    cnt = d.sum(axis=1)                                   # [n, c_out]
    keep = cnt.astype(np.float32) >= np.float32(tau) * np.float32(s.ho * s.wo)
    d_eff = d & keep[:, None, :]
    got = O.unpack_mask(res.mask, s.c_out).reshape(d.shape)
    np.testing.assert_array_equal(got, d_eff)
    assert res.channels_skipped == int((~keep).sum())
    assert res.active == int(d_eff.sum()) and res.cond_macs == res.active * s.kh * s.kw * s.c_r
    # kept channels are untouched, dropped ones equal the base-path-only layer
    base = O.gated_conv(s, x, wb, wc, bn, np.full(s.c_out, INF, np.float32))
    ky = np.broadcast_to(keep[:, None, None, :], res.y.shape)
    np.testing.assert_array_equal(res.y[ky], plain.y[ky])
    np.testing.assert_array_equal(res.y[~ky], base.y[~ky])
    assert 0 < res.channels_skipped < res.channels


def test_channel_gate_is_per_image():
    """Eq. 4 sums over one feature map: an image's decision does not depend on its batch."""
    s2 = O.Shape(2, 6, 6, 8, 8, groups=2)
    x, wb, wc, bn = make_layer(("cg-img", 8), s2)
    delta = np.full(8, 0.2, np.float32)
    both = O.gated_conv(s2, x, wb, wc, bn, delta, channel_tau=0.45)
    s1 = O.Shape(1, 6, 6, 8, 8, groups=2)
    for i in range(2):
        one = O.gated_conv(s1, x[i:i + 1], wb, wc, bn, delta, channel_tau=0.45)
        np.testing.assert_array_equal(one.y[0], both.y[i])


# --------------------------------------------------------------------------- channel reordering
def test_reordering_output_channels_only_relabels_the_layer():
    """A layer whose output channels are gathered by a permutation gives the permuted outputs and
    mask bits of the original layer, and a consumer whose input channels are gathered the same way
    (ungated, so that its split does not move) gives its original output."""
    from paper_1805_12549_b200 import permute, synth
    s = O.Shape(2, 6, 6, 16, 32, 3, 3, 1, 1, 4)
    key = ("permute", 1)
    x = synth.smoothed_noise((key, "x"), s.n, s.h, s.w, s.c_in)
    wb, wc = synth.kaiming_weights(key, s.c_out, 3, 3, s.c_in, s.groups)
    bn = synth.bn_params(key, s.c_out)
    delta = synth.rng(key, "delta").normal(0.3, 0.5, s.c_out).astype(np.float32)
    ref = O.gated_conv(s, x, wb, wc, bn, delta)
    d = permute.unpack_mask(ref.mask, s.c_out)
    np.testing.assert_array_equal(d, O.unpack_mask(ref.mask, s.c_out))
    perm = permute.order_by_firing_rate(d)
    assert sorted(perm.tolist()) == list(range(s.c_out))
    rates = d.mean(0)[perm]
    assert (np.diff(rates) <= 1e-12).all()
    wb2, wc2, pc = permute.permute_output_channels(wb, wc, {**bn, "delta": delta}, perm)
    delta2 = pc.pop("delta")
    got = O.gated_conv(s, x, wb2, wc2, pc, delta2)
    np.testing.assert_array_equal(got.y, ref.y[..., perm])
    np.testing.assert_array_equal(O.unpack_mask(got.mask, s.c_out), d[:, perm])
    # consumer: an ungated 1x1 layer over the 32 channels
    s2 = O.Shape(2, 6, 6, 32, 8, 1, 1, 1, 0, 1)
    w2, _ = synth.kaiming_weights((key, "next"), 8, 1, 1, 32, 1)
    bn2 = synth.bn_params((key, "next"), 8)
    shut = np.full(8, np.inf, np.float32)
    empty = np.zeros((8, 1, 1, 0), np.float32)
    a = O.gated_conv(s2, ref.y, w2, empty, bn2, shut)
    w2p, w2c = permute.permute_input_channels(w2, perm, 1)
    assert w2c.size == 0
    b = O.gated_conv(s2, got.y, w2p, w2c, bn2, shut)
    np.testing.assert_allclose(b.y, a.y, rtol=0, atol=1e-5)     # same products, summed in another order


# --------------------------------------------------------------------------- two-sided gate
@pytest.mark.parametrize("s", SHAPES[:3])
def test_two_sided_gate_keeps_the_band_between_the_thresholds(s):
    """Section 3.2: s(x, Delta_h, Delta_l) = theta(Delta_h - x) o theta(x - Delta_l).  An
    activation takes Eq. 1's second case iff its normalised partial sum lies in
    [Delta_l, Delta_h]; decided here from the library partial sums (away from near-ties)."""
    x, wb, wc, bn = make_layer(("band", s.c_in, s.h), s)
    g = synth.rng("band-delta", s.c_in)
    lo = g.uniform(-0.8, 0.0, s.c_out).astype(np.float32)
    hi = (lo + g.uniform(0.3, 1.2, s.c_out)).astype(np.float32)
    res = O.gated_conv(s, x, wb, wc, bn, lo, delta_high=hi)
    p_ref = lib_conv64(x[..., :s.c_p], wb, s.stride, s.pad)
    full_ref = lib_conv64(x, np.concatenate([wb, wc], axis=3), s.stride, s.pad)
    sg = np.sqrt(bn["gate_var"].astype(np.float64) + s.bn_eps)
    t_lo = lo.astype(np.float64) * sg + bn["gate_mean"].astype(np.float64)
    t_hi = hi.astype(np.float64) * sg + bn["gate_mean"].astype(np.float64)
    d_ref = (p_ref >= t_lo) & (p_ref <= t_hi)
    clear = (np.abs(p_ref - t_lo) > 1e-4) & (np.abs(p_ref - t_hi) > 1e-4)
    d = O.unpack_mask(res.mask, s.c_out).reshape(p_ref.shape)
    assert (d == d_ref)[clear].all()
    y_ref = np.where(d, bn_relu64(full_ref, bn["gamma"], bn["beta"], bn["mean_full"], bn["var_full"], s.bn_eps),
                     bn_relu64(p_ref, bn["gamma"], bn["beta"], bn["mean_base"], bn["var_base"], s.bn_eps))
    np.testing.assert_allclose(res.y, y_ref, rtol=1e-5, atol=1e-5)
    one_sided = O.gated_conv(s, x, wb, wc, bn, lo)
    assert 0 < res.active < one_sided.active, "the upper threshold must shut some gates"
    assert res.active == int(d.sum())
    assert res.cond_macs == s.kh * s.kw * s.c_r * res.active


def test_two_sided_gate_limits_and_ties():
    """Delta_h = +inf is the one-sided gate; Delta_h below Delta_l shuts everything; a partial sum
    equal to the upper threshold still fires (theta(0) = 1), the next float above does not; the
    normalise-then-compare form agrees with the merged one away from ties."""
    s = O.Shape(1, 6, 6, 8, 8, groups=4)
    x, wb, wc, bn = make_layer(("band2", 1), s)
    lo = np.full(s.c_out, -0.2, np.float32)
    one = O.gated_conv(s, x, wb, wc, bn, lo)
    same = O.gated_conv(s, x, wb, wc, bn, lo, delta_high=np.full(s.c_out, INF, np.float32))
    np.testing.assert_array_equal(one.mask, same.mask)
    np.testing.assert_array_equal(one.y, same.y)
    none = O.gated_conv(s, x, wb, wc, bn, lo, delta_high=np.full(s.c_out, -0.5, np.float32))
    assert none.active == 0
    # exact tie at the upper threshold: unit statistics, eps = 0, Delta_h = a partial sum itself
    s0 = O.Shape(1, 6, 6, 8, 8, groups=4, bn_eps=0.0)
    bn0 = dict(bn, gate_mean=np.zeros(s.c_out, np.float32), gate_var=np.ones(s.c_out, np.float32))
    shut = np.full(s.c_out, -INF, np.float32)
    p = O.gated_conv(s0, x, wb, wc, bn0, shut).p.reshape(-1, s.c_out)
    hi = p[7].copy()                                   # pixel 7's partial sums as upper thresholds
    tie = O.gated_conv(s0, x, wb, wc, bn0, shut, delta_high=hi)
    assert O.unpack_mask(tie.mask, s.c_out)[7].all()
    below = O.gated_conv(s0, x, wb, wc, bn0, shut, delta_high=np.nextafter(hi, np.float32(-INF)))
    assert not O.unpack_mask(below.mask, s.c_out)[7].any()
    merged = O.gated_conv(s, x, wb, wc, bn, lo, delta_high=lo + np.float32(0.7))
    split = O.gated_conv(s, x, wb, wc, bn, lo, delta_high=lo + np.float32(0.7), gate_form=1)
    assert (O.unpack_mask(merged.mask, s.c_out) != O.unpack_mask(split.mask, s.c_out)).sum() <= 2
