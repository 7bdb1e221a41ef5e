"""CG-ResNet-18 over the C ABI: the glue operators against their definitions, every layer of a
two-image forward pass against the oracle fed with that layer's own input, and the FLOP model of
the whole network (Section 3.1) at the target density and with every gate open."""
import numpy as np
import pytest

from oracle import oracle as O
from tests import cases

pytestmark = pytest.mark.gpu


def _f32(t):
    return t.float().cpu().numpy()


def _bf16_dev(a):
    return cases._to_dev(np.ascontiguousarray(a, np.float32), "bf16")


def _rand_bf16(key, shape):
    from paper_1805_12549_b200 import synth
    return synth.bf16_round(synth.rng("net_ops", key).standard_normal(shape, dtype=np.float32))


@pytest.mark.parametrize("n,h,w,c,k,stride,pad,k_pad", [(2, 13, 11, 3, 7, 2, 3, 152), (3, 20, 18, 3, 7, 2, 3, 192),
                                                       (2, 9, 10, 4, 3, 1, 1, 40), (1, 8, 8, 3, 7, 2, 2, 152)])
def test_im2col_matches_the_patch_definition(n, h, w, c, k, stride, pad, k_pad):
    import torch
    from paper_1805_12549_b200 import binding as B
    x = _rand_bf16("im2col", (n, h, w, c))
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    ref = np.zeros((n, ho, wo, k_pad), np.float32)
    xp = np.zeros((n, h + 2 * pad, w + 2 * pad, c), np.float32)
    xp[:, pad:pad + h, pad:pad + w] = x
    for i in range(ho):
        for j in range(wo):
            ref[:, i, j, :k * k * c] = xp[:, i * stride:i * stride + k, j * stride:j * stride + k].reshape(n, -1)
    a = torch.full((n, ho, wo, k_pad), 7.0, dtype=torch.bfloat16, device="cuda")
    B.cg_im2col_bf16(_bf16_dev(x), a, k, stride, pad)
    np.testing.assert_array_equal(_f32(a), ref)


def test_subsample_maxpool_avgpool_match_their_definitions():
    import torch
    from paper_1805_12549_b200 import binding as B, synth
    n, h, w, c = 3, 9, 14, 24
    x = _rand_bf16("pool", (n, h, w, c))
    xd = _bf16_dev(x)
    y = torch.empty((n, 5, 7, c), dtype=torch.bfloat16, device="cuda")
    B.cg_subsample_bf16(xd, y, 2)
    np.testing.assert_array_equal(_f32(y), x[:, ::2, ::2])
    ho, wo = (h + 2 - 3) // 2 + 1, (w + 2 - 3) // 2 + 1
    xp = np.full((n, h + 2, w + 2, c), -np.inf, np.float32)
    xp[:, 1:-1, 1:-1] = x
    ref = np.stack([np.stack([xp[:, 2 * i:2 * i + 3, 2 * j:2 * j + 3].max((1, 2)) for j in range(wo)], 1)
                    for i in range(ho)], 1)
    y = torch.empty((n, ho, wo, c), dtype=torch.bfloat16, device="cuda")
    B.cg_maxpool_bf16(xd, y, 3, 2, 1)
    np.testing.assert_array_equal(_f32(y), ref)
    y = torch.empty((n, 1, 1, c), dtype=torch.bfloat16, device="cuda")
    B.cg_avgpool_bf16(xd, y)
    mean = x.reshape(n, h * w, c).astype(np.float64).mean(1)
    got = _f32(y).reshape(n, c)
    assert np.abs(got - mean).max() <= 2.0 ** -8 * np.abs(mean).max() + 1e-6   # one bf16 rounding of an fp32 sum


@pytest.fixture(scope="module")
def network():
    import torch
    from paper_1805_12549_b200 import resnet18 as R
    net = R.CgResNet18(groups=4)
    gated, other = net.macs_per_image()
    tau = R.density_for_reduction(2.8, 4, gated, other)
    x = R.synthetic_images("test_resnet18", 4)
    net.calibrate(x, tau)
    torch.cuda.synchronize()
    return net, x, tau


def test_flop_budget(network):
    net, _, tau = network
    gated, other = net.macs_per_image()
    assert len(net.gated_specs) == 16
    assert abs((gated + other) / 1e9 - 1.814) < 0.01     # multiplications of ResNet-18 at 224 x 224
    assert abs(tau - 0.072) < 0.005                      # density that gives 2.8x with G = 4


def test_every_layer_matches_the_oracle_on_two_images(network):
    import torch
    from paper_1805_12549_b200 import synth
    net, x, _ = network
    inst = net.instance(2)
    record = []
    logits = inst.forward(x[:2].contiguous(), record=record)
    torch.cuda.synchronize()
    per, summary = inst.stats()
    assert all(st.device_status == 0 for st in per.values())
    assert torch.isfinite(logits.float()).all()
    assert len(record) == len(net.specs) == 21
    exempt = 0
    for s, xin, res, y, mask in record:
        bn = {k: v.cpu().numpy() for k, v in s.params.items()}
        delta = s.delta.cpu().numpy()
        wb = _f32(s.wb)
        wc = _f32(s.wc) if s.wc is not None else np.zeros((s.c_out, s.k, s.k, 0), np.float32)
        if s.name == "stem":
            # the definition: a 7x7 stride-2 convolution of the image (the patch matrix is the GPU's business)
            shape = O.Shape(2, net.image, net.image, 3, s.c_out, 7, 7, 2, 3, 1, 1e-5, 1)
            xin_np, wb = _f32(x[:2]), synth.bf16_round(net.stem_filter)
        else:
            shape = O.Shape(2, s.h, s.h, s.c_in, s.c_out, s.k, s.k, s.stride, s.pad, s.groups, 1e-5, int(s.relu))
            xin_np = _f32(xin)
        ref = O.gated_conv(shape, xin_np, wb, wc, bn, delta, None if res is None else _f32(res), out_bf16=True)
        c = cases.Case(s.name, shape, "bf16", xin_np, wb, wc, bn, delta)
        m = mask.cpu().numpy().view(np.uint32) if mask is not None else ref.mask
        if s.gated:
            exempt += cases.compare(c, ref, _f32(y), m, None)
        else:
            assert ref.active == 0                       # Delta = +inf: the base path is the layer
            err = np.abs(_f32(y).astype(np.float64) - ref.y)
            assert (err <= cases.BF16_ATOL + cases.BF16_RTOL * np.abs(ref.y)).all(), s.name
    assert exempt <= 64                                  # gate flips within 1e-3 of Delta, whole network
    inst.close()


def test_flop_reduction_and_density_one_twin(network):
    import torch
    net, x, tau = network
    inst = net.instance(4)
    inst.forward(x)
    torch.cuda.synchronize()
    _, at_target = inst.stats()
    assert abs(at_target["gated_layer_density"] - tau) < 0.01     # calibrated on these images
    assert abs(at_target["flop_reduction"] - 2.8) < 0.15
    y_target = inst.forward(x).float().clone()
    inst.stats()                                         # (reading clears the counters)
    net.set_density(1.0)
    y_dense = inst.forward(x).float().clone()
    torch.cuda.synchronize()
    _, dense = inst.stats()
    net.set_density(tau)
    assert dense["gated_layer_density"] > 0.999
    assert abs(dense["flop_reduction"] - 1.0) < 1e-3
    assert torch.isfinite(y_dense).all() and torch.isfinite(y_target).all()
    assert inst.launches_per_forward() >= 21 + 6
    inst.close()
