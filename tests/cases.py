"""Shared helpers of the parity tests: build a seeded case, run the oracle, run the CUDA
library through its C ABI, compare with the stated tolerances."""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from oracle import oracle as O
from paper_1805_12549_b200 import synth

INF = float("inf")

# bf16 tolerance of the layer outputs (fp32 accumulation over the same bf16-rounded inputs)
BF16_ATOL, BF16_RTOL = 2e-2, 1e-2
# an activation whose normalised partial sum is this close to Delta may flip its gate
NEAR_TIE = 1e-3


@dataclass
class Case:
    name: str
    s: O.Shape
    dtype: str                  # "f32" | "bf16" | "i8"
    x: np.ndarray
    wb: np.ndarray
    wc: np.ndarray
    bn: dict = field(default_factory=dict)       # float params (f32/bf16) or q_* params (i8)
    delta: np.ndarray | None = None
    residual: np.ndarray | None = None
    shift: int = 0
    grouped: bool = False
    channel_tau: float = 0.0    # tau_c of the channel-wise gate (Eq. 4); 0 = off
    delta_high: np.ndarray | None = None   # upper thresholds of the two-sided gate (Section 3.2)


def _quantile_delta(p_hat: np.ndarray, density: float) -> float:
    """Scalar Delta such that the fraction of p_hat >= Delta is `density`."""
    if density >= 1.0:
        return -INF
    if density <= 0.0:
        return INF
    return float(np.quantile(p_hat.astype(np.float64), 1.0 - density))


def make_float_case(name, s: O.Shape, dtype="bf16", density=0.3, delta=None, rho=0.0,
                    calib_images=4, separate=True, residual=False, smooth=True,
                    grouped=False) -> Case:
    """Seeded layer.  Gate statistics are the per-channel mean/variance of the oracle's partial
    sums over the first `calib_images` images; Delta is one scalar per layer, the quantile of the
    normalised partial sums that gives `density` (unless `delta` is given)."""
    key = (name, s.n, s.h, s.w, s.c_in, s.c_out, s.stride, s.groups)
    if smooth:
        x = synth.smoothed_noise((key, "x"), s.n, s.h, s.w, s.c_in, rho=rho)
    else:
        x = synth.rng(key, "x").standard_normal((s.n, s.h, s.w, s.c_in), dtype=np.float32)
    wb, wc = synth.kaiming_weights(key, s.c_out, s.kh, s.kw, s.c_in, s.groups)
    if dtype == "bf16":
        x, wb, wc = synth.bf16_round(x), synth.bf16_round(wb), synth.bf16_round(wc)
    bn = synth.bn_params(key, s.c_out, separate=separate)
    res = None
    if residual:
        res = synth.residual(key, (s.n, s.ho, s.wo, s.c_out))
        if dtype == "bf16":
            res = synth.bf16_round(res)
    if delta is None:
        nc = max(1, min(calib_images, s.n))
        sc = O.Shape(**{**s.__dict__, "n": nc})
        probe = O.gated_conv(sc, x[:nc], wb, wc, bn, np.full(s.c_out, INF, np.float32),
                             grouped=grouped)
        p = probe.p.reshape(-1, s.c_out).astype(np.float64)
        bn["gate_mean"] = p.mean(axis=0).astype(np.float32)
        bn["gate_var"] = np.maximum(p.var(axis=0), 1e-6).astype(np.float32)
        p_hat = (p - bn["gate_mean"]) / np.sqrt(bn["gate_var"].astype(np.float64) + s.bn_eps)
        delta = np.full(s.c_out, _quantile_delta(p_hat, density), np.float32)
    else:
        delta = np.broadcast_to(np.asarray(delta, np.float32), (s.c_out,)).copy()
    return Case(name, s, dtype, x, wb, wc, bn, delta, res, 0, grouped)


def make_int8_case(name, s: O.Shape, density=0.3, shift=24, calib_images=4) -> Case:
    key = (name, "i8", s.n, s.h, s.w, s.c_in, s.c_out, s.stride, s.groups)
    x = synth.int8_activations(key, s.n, s.h, s.w, s.c_in)
    wb, wc = synth.int8_weights(key, s.c_out, s.kh, s.kw, s.c_in, s.groups)
    nc = max(1, min(calib_images, s.n))
    sc = O.Shape(**{**s.__dict__, "n": nc})
    q0 = {"q_gate_thr": np.full(s.c_out, np.iinfo(np.int32).min, np.int32),
          "q_mul_base": np.ones(s.c_out, np.int32), "q_mul_full": np.ones(s.c_out, np.int32),
          "q_off_base": np.zeros(s.c_out, np.int64), "q_off_full": np.zeros(s.c_out, np.int64)}
    # all-open run with unit scale and a shift of 1 is only used for its partial sums
    probe = O.gated_conv_i8(sc, 1, x[:nc], wb, wc, q0)
    p = probe.p.reshape(-1, s.c_out).astype(np.float64)
    # full sums via a second all-open pass are not exposed; estimate sigma_full from variances:
    # R has (G-1) times the terms of P with the same statistics
    sigma_base = p.std() + 1.0
    sigma_full = sigma_base * np.sqrt(s.groups)
    q = synth.int8_requant(key, s.c_out, shift, sigma_base, sigma_full)
    if density >= 1.0:
        q["q_gate_thr"] = np.full(s.c_out, np.iinfo(np.int32).min, np.int32)
    elif density <= 0.0:
        q["q_gate_thr"] = np.full(s.c_out, np.iinfo(np.int32).max, np.int32)
    else:
        q["q_gate_thr"] = np.ceil(np.quantile(p, 1.0 - density, axis=0)).astype(np.int32)
    return Case(name, s, "i8", x, wb, wc, q, None, None, shift)


def run_oracle(c: Case, **kw) -> O.Result:
    if c.dtype == "i8":
        return O.gated_conv_i8(c.s, c.shift, c.x, c.wb, c.wc, c.bn)
    return O.gated_conv(c.s, c.x, c.wb, c.wc, c.bn, c.delta, c.residual,
                        out_bf16=(c.dtype == "bf16"), grouped=c.grouped,
                        channel_tau=c.channel_tau, delta_high=c.delta_high, **kw)


# ----------------------------------------------------------------------------- GPU side
def _to_dev(a, dtype):
    import torch
    if a is None:
        return None
    if dtype == "bf16":
        bits = synth.bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    if dtype == "i8":
        return torch.from_numpy(np.ascontiguousarray(a, np.int8)).cuda()
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).cuda()


class GpuCase:
    """Device copies of a Case plus a handle; run() calls cg_conv_forward through the C ABI."""

    def __init__(self, c: Case, algo=0, cond_mode=0):
        import torch
        from paper_1805_12549_b200 import binding as B
        self.B, self.torch, self.c = B, torch, c
        s = c.s
        dt = {"f32": B.CG_F32, "bf16": B.CG_BF16, "i8": B.CG_I8}[c.dtype]
        self.conv = B.GatedConv(s.n, s.h, s.w, s.c_in, s.c_out, k=s.kh, stride=s.stride, pad=s.pad,
                                groups=s.groups, dtype=dt, bn_eps=s.bn_eps, relu=bool(s.relu),
                                has_residual=c.residual is not None, requant_shift=c.shift,
                                algo=algo, cond_mode=cond_mode, grouping=c.grouped,
                                channel_tau=c.channel_tau)
        self.x = _to_dev(c.x, c.dtype)
        self.wb = _to_dev(c.wb, c.dtype)
        self.wc = _to_dev(c.wc, c.dtype)
        self.res = _to_dev(c.residual, c.dtype)
        self.params = {}
        for k, v in c.bn.items():
            if v is None:
                continue
            self.params[k] = torch.from_numpy(np.ascontiguousarray(v)).cuda()
        if c.delta_high is not None:
            self.params["delta_high"] = torch.from_numpy(np.ascontiguousarray(c.delta_high, np.float32)).cuda()
        self.bn = B.make_bn(self.params)
        self.delta = None if c.delta is None else torch.from_numpy(c.delta).cuda()
        # y, mask and the workspace sit inside larger buffers whose margins hold a known pattern:
        # a kernel that writes outside its tensors is caught by check_guards() after every run
        self.y, self._y_buf = self._guarded(self.conv.desc.n * self.conv.ho * self.conv.wo * s.c_out,
                                            self.B._TORCH_DTYPE[dt])
        self.y = self.y.view(self.conv.desc.n, self.conv.ho, self.conv.wo, s.c_out)
        self.mask, self._m_buf = self._guarded(self.conv.m * self.conv.words, torch.int32)
        self.mask = self.mask.view(self.conv.m, self.conv.words)
        self._ws_buf = None
        if self.conv.workspace is not None:
            n = self.conv.workspace.numel()
            ws, self._ws_buf = self._guarded(n, torch.uint8)
            self.conv.workspace = ws

    GUARD = 4096      # bytes of pattern before and after each tensor
    PATTERN = 0x5A

    def _guarded(self, numel, dtype):
        torch = self.torch
        esz = torch.empty(0, dtype=dtype).element_size()
        nbytes = numel * esz
        pad = (-nbytes) % 256
        buf = torch.full((self.GUARD + nbytes + pad + self.GUARD,), self.PATTERN, dtype=torch.uint8, device="cuda")
        inner = buf[self.GUARD:self.GUARD + nbytes].view(dtype)
        return inner, buf

    def check_guards(self):
        for name, buf, t in (("y", self._y_buf, self.y), ("mask", self._m_buf, self.mask),
                             ("workspace", self._ws_buf, self.conv.workspace)):
            if buf is None:
                continue
            nbytes = t.numel() * t.element_size()
            head = buf[:self.GUARD]
            tail = buf[self.GUARD + nbytes:]
            assert bool((head == self.PATTERN).all()), f"write in front of {name}"
            assert bool((tail == self.PATTERN).all()), f"write behind {name}"

    def run(self, with_mask=True):
        self.y.fill_(0)
        self.mask.fill_(-1)
        self.conv.forward(self.x, self.wb, self.wc, self.bn, self.delta, self.y,
                          self.mask if with_mask else None, self.res)
        st = self.conv.stats()
        self.torch.cuda.synchronize()
        self.check_guards()
        y = self.y.float().cpu().numpy() if self.c.dtype != "i8" else self.y.cpu().numpy()
        mask = self.mask.cpu().numpy().view(np.uint32)
        return y, mask, st

    def close(self):
        self.conv.close()


def compare(c: Case, ref: O.Result, y, mask, st, exact=False):
    """Parity bars.  exact=True (direct path, int8): bit-exact masks and outputs.
    Otherwise (bf16 tensor-core path): masks equal except where the oracle's normalised partial
    sum is within NEAR_TIE of Delta; outputs within BF16_ATOL + BF16_RTOL*|ref| wherever the
    masks agree.  Returns the number of exempt (near-tie) mismatches."""
    s = c.s
    assert y.shape == ref.y.shape
    d_ref = O.unpack_mask(ref.mask, s.c_out)
    d_gpu = O.unpack_mask(mask, s.c_out)
    if s.c_out % 32:
        assert (mask[:, -1] >> np.uint32(s.c_out % 32)).max() == 0, "padding bits must be zero"
    if exact or c.dtype == "i8":
        np.testing.assert_array_equal(mask, ref.mask)
        if c.dtype == "i8":
            np.testing.assert_array_equal(y, ref.y)
        else:
            np.testing.assert_array_equal(y.view(np.uint32), ref.y.view(np.uint32))
        exempt = 0
    else:
        gm = c.bn.get("gate_mean", c.bn["mean_base"]) if c.bn.get("gate_mean") is not None \
            else c.bn["mean_base"]
        gv = c.bn.get("gate_var", c.bn["var_base"]) if c.bn.get("gate_var") is not None \
            else c.bn["var_base"]
        p = ref.p.reshape(-1, s.c_out).astype(np.float64)
        with np.errstate(invalid="ignore"):
            p_hat = (p - gm) / np.sqrt(gv.astype(np.float64) + s.bn_eps)
            near = np.abs(p_hat - c.delta.astype(np.float64)) < NEAR_TIE
            if c.delta_high is not None:      # two-sided gate: a tie at either threshold may flip
                near |= np.abs(p_hat - c.delta_high.astype(np.float64)) < NEAR_TIE
        diff = d_ref != d_gpu
        bad = diff & ~near
        assert not bad.any(), f"{int(bad.sum())} gate decisions differ away from the threshold"
        exempt = int(diff.sum())
        agree = ~diff.reshape(ref.y.shape)
        err = np.abs(y.astype(np.float64) - ref.y)
        tol = BF16_ATOL + BF16_RTOL * np.abs(ref.y)
        worst = (err - tol)[agree].max() if agree.any() else -1.0
        assert worst <= 0, f"output error exceeds tolerance by {worst}"
    if st is not None:
        assert st.outputs == ref.outputs
        assert st.active == int(d_gpu.sum())
        assert st.dense_macs == ref.dense_macs
        k2 = s.kh * s.kw
        assert st.gated_macs == k2 * (s.c_p * st.outputs + s.c_r * st.active)
        assert st.executed_macs >= st.gated_macs
        assert st.device_status == 0
    return exempt
