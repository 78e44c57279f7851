"""Pins for the oracle's AdaRMSNorm (Eq. 2, App. B.3) and Euler flow update (Sec. 2.1, App. C)."""
import numpy as np
import pytest
import torch

from oracle import reflex_oracle as orc
from paper_2607_14695_b200 import synth


def _params(rng, D, Cd, Hd, std=0.3):
    return (rng.standard_normal((Hd, Cd)).astype(np.float32) * np.float32(std), rng.standard_normal(Hd).astype(np.float32) * np.float32(std),
            rng.standard_normal((D, Hd)).astype(np.float32) * np.float32(std), rng.standard_normal(D).astype(np.float32) * np.float32(std))


@pytest.mark.parametrize("eps", [1e-6, 1e-5])
def test_gate_off_reduces_to_plain_rmsnorm(eps):
    """gamma = 1 + MLP(c); MLP(c) = 0 when W2 = 0, b2 = 0 (any c), or when b1 = b2 = 0 and c = 0
    (SiLU(0) = 0). Then AdaRMSNorm is weight-free RMSNorm == torch.nn.functional.rms_norm in fp64."""
    rng = np.random.default_rng(0)
    R, D, Cd, Hd = 5, 48, 6, 7
    x = rng.standard_normal((R, D)).astype(np.float32) * 3
    W1, b1, W2, b2 = _params(rng, D, Cd, Hd)
    c = rng.standard_normal(Cd).astype(np.float32)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (D,), eps=eps).numpy()
    hand = x.astype(np.float64) / np.sqrt((x.astype(np.float64) ** 2).mean(-1, keepdims=True) + eps)
    y1, g1 = orc.adarmsnorm(x, c, W1, b1, np.zeros_like(W2), np.zeros_like(b2), eps, return_gate=True)
    y2, g2 = orc.adarmsnorm(x, np.zeros_like(c), W1, np.zeros_like(b1), W2, np.zeros_like(b2), eps, return_gate=True)
    for y, g in ((y1, g1), (y2, g2)):
        assert np.array_equal(g, np.ones(D))
        assert np.max(np.abs(y - ref)) <= 1e-12 and np.max(np.abs(y - hand)) <= 1e-12


def test_gate_hand_computed_scalar_mlp():
    """Cd = Hd = 1: gamma_i = 1 + W2_i * silu(w*c + b) + b2_i with silu(z) = z / (1 + e^-z) worked by hand."""
    w, b, c = 0.5, 0.25, 2.0
    z = w * c + b                       # 1.25
    silu = z / (1.0 + np.exp(-z))
    W2 = np.array([[2.0], [-1.0], [0.0]], np.float32); b2 = np.array([0.5, 0.0, -0.25], np.float32)
    x = np.array([[3.0, 4.0, 0.0]], np.float32)     # mean square = 25/3
    y, g = orc.adarmsnorm(x, np.array([c], np.float32), np.array([[w]], np.float32), np.array([b], np.float32), W2, b2, 0.0, return_gate=True)
    want_g = np.array([1 + 2 * silu + 0.5, 1 - silu, 0.75])
    assert np.max(np.abs(g - want_g)) <= 1e-15
    r = np.sqrt(25.0 / 3.0)
    assert np.max(np.abs(y[0] - np.array([3 / r, 4 / r, 0.0]) * want_g)) <= 1e-15


def test_gate_matches_torch_mlp_fp64():
    """gamma == 1 + Linear(SiLU(Linear(c))) from torch.nn.functional in fp64 (library routine as checker)."""
    rng = np.random.default_rng(1)
    R, D, Cd, Hd = 3, 40, 12, 9
    W1, b1, W2, b2 = _params(rng, D, Cd, Hd)
    c = rng.standard_normal(Cd).astype(np.float32); x = rng.standard_normal((R, D)).astype(np.float32)
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(a).double()
    gate = 1 + F.linear(F.silu(F.linear(t(c), t(W1), t(b1))), t(W2), t(b2))
    want = F.rms_norm(t(x), (D,), eps=1e-6) * gate
    y, g = orc.adarmsnorm(x, c, W1, b1, W2, b2, 1e-6, return_gate=True)
    assert np.max(np.abs(g - gate.numpy())) <= 1e-13 and np.max(np.abs(y - want.numpy())) <= 1e-12


def test_norm_invariants():
    rng = np.random.default_rng(2)
    R, D, Cd, Hd = 6, 64, 5, 4
    W1, b1, W2, b2 = _params(rng, D, Cd, Hd)
    c = rng.standard_normal(Cd).astype(np.float32)
    x = rng.standard_normal((R, D)).astype(np.float32)
    x[3] = 0.0
    eps = 1e-6
    y, g = orc.adarmsnorm(x, c, W1, b1, W2, b2, eps, return_gate=True)
    ms = (x.astype(np.float64) ** 2).mean(-1)
    assert np.allclose(((y / g) ** 2).mean(-1), ms / (ms + eps), rtol=0, atol=1e-12)   # mean((y/gamma)^2) = ms/(ms+eps)
    assert np.array_equal(y[3], np.zeros(D))                                            # zero row stays finite zero
    xs = np.delete(x, 3, axis=0)
    y0 = orc.adarmsnorm(xs, c, W1, b1, W2, b2, 0.0)
    assert np.allclose(((y0 / g) ** 2).mean(-1), 1.0, rtol=0, atol=1e-12)               # eps = 0: unit RMS
    y4 = orc.adarmsnorm((xs * np.float32(4.0)).astype(np.float32), c, W1, b1, W2, b2, 0.0)
    assert np.max(np.abs(y4 - y0)) <= 1e-12                                             # scale invariance, eps = 0
    # per-stream gates in the batched form
    cond = rng.standard_normal((2, Cd)).astype(np.float32)
    yb = orc.adarmsnorm_batched(np.stack([x, x]), cond, W1, b1, W2, b2, eps)
    assert np.array_equal(yb[0], orc.adarmsnorm(x, cond[0], W1, b1, W2, b2, eps))
    assert not np.array_equal(yb[0], yb[1])


def test_outlier_rows_stay_finite_and_bf16_rounding_budget():
    """Stress input of the long-context config: N(0,1) with x1e3 outliers. The oracle's double result,
    rounded to bf16, differs from itself by at most half a bf16 ulp: the tolerance budget belongs to the
    GPU path (max(2e-2, 2^-7 |y|) leaves more than 2x room)."""
    w = synth.CONFIGS["cfg5"].with_(B=2)
    x = synth.norm_input(w, 0, 0)
    W1, b1, W2, b2 = synth.gate_weights(w, 0)
    for t in (0.0, 1e-4, 1.0 - 1e-4, 1.0):
        cond = synth.cond_vectors(w, t)
        y = orc.adarmsnorm_batched(x, cond, W1, b1, W2, b2, 1e-6)
        assert np.isfinite(y).all()
        yr = synth.round_storage(y.astype(np.float32), synth.DTYPE_BF16).astype(np.float64)
        assert (np.abs(yr - y) <= np.maximum(2e-2, 2.0 ** -7 * np.abs(y)) * 0.51).all()
    assert (np.abs(x) > 100).sum() > 0


def test_flow_closed_forms():
    rng = np.random.default_rng(3)
    n = 50
    for K in (1, 4, 10):
        x0 = rng.standard_normal(n)
        v = rng.standard_normal(n).astype(np.float32)
        x = x0.copy()
        for k in range(K):
            orc.flow_step(x, v, K)
        assert np.max(np.abs(x - (x0 - v.astype(np.float64)))) <= 1e-14          # constant v: x_K = x_0 - v
        x = x0.astype(np.float32).astype(np.float64); start = x.copy()
        for k in range(K):
            orc.flow_step(x, x.astype(np.float32), K)                             # v = x (fp32 copy of the state)
        assert np.max(np.abs(x - start * (1 - 1.0 / K) ** K)) <= 1e-6
        # straight path x_t = t*eps + (1-t)*a has velocity eps - a: Euler lands on a exactly
        eps_ = rng.standard_normal(n).astype(np.float32); a = rng.standard_normal(n).astype(np.float32)
        vel = (eps_.astype(np.float64) - a.astype(np.float64)).astype(np.float32)
        x = vel.astype(np.float64) + a.astype(np.float64)                         # state at t = 1
        for k in range(K):
            orc.flow_step(x, vel, K)
        assert np.max(np.abs(x - a)) <= 1e-14
        assert orc.flow_time(0, K) == 1.0 and orc.flow_time(K, K) == 0.0
        assert all(abs(orc.flow_time(k, K) - (K - k) / K) < 1e-16 for k in range(K + 1))


def test_bf16_rounding_helper_is_rne():
    """The shared input rounding is round-to-nearest-even, same as torch's float32 -> bfloat16 cast."""
    rng = np.random.default_rng(4)
    a = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 50, np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38], np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    assert np.array_equal(synth.round_storage(a, synth.DTYPE_BF16), want)
    bits = synth.f32_to_bf16_bits(a)
    assert np.array_equal(torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float().numpy(), want)
