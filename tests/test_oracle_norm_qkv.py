"""Pins for the oracle's adaptive norm + packed Q/K/V projection (Sec. 3.3 "System Optimizations": W_QKV = [W_Q; W_K; W_V];
Sec. 4 "Operator Fusion Impact": the norm combined with the linear layer after it)."""
import numpy as np
import torch

from oracle import reflex_oracle as orc


def _mlp(rng, D, Cd, Hd, std=0.3):
    return (rng.standard_normal((Hd, Cd)).astype(np.float32) * np.float32(std), rng.standard_normal(Hd).astype(np.float32) * np.float32(std),
            rng.standard_normal((D, Hd)).astype(np.float32) * np.float32(std), rng.standard_normal(D).astype(np.float32) * np.float32(std))


def test_hand_worked_example():
    """One row, D = 2, gate off: x = (3, 4), mean square 12.5, y = x / sqrt(12.5). Q weights (1, 0) and (0, 2), K weight (1, 1),
    V weight (1, -1): q = (y0, 2 y1), k = y0 + y1, v = y0 - y1."""
    x = np.array([[3.0, 4.0]], np.float32)
    z1 = np.zeros((1, 1), np.float32); zb = np.zeros(1, np.float32)
    W = np.array([[1, 0], [0, 2], [1, 1], [1, -1]], np.float32)
    q, k, v = orc.adarmsnorm_qkv(x, np.zeros(1, np.float32), z1, zb, np.zeros((2, 1), np.float32), np.zeros(2, np.float32), W, Hq=2, Hkv=1, d=1, eps=0.0)
    r = np.sqrt(12.5)
    assert np.allclose(q[0, :, 0], [3 / r, 8 / r], rtol=0, atol=1e-15)
    assert abs(k[0, 0, 0] - 7 / r) <= 1e-15 and abs(v[0, 0, 0] + 1 / r) <= 1e-15


def test_identity_weights_return_the_norm_output():
    """W_QKV = [I; I; I] with Hq = Hkv = 1, d = D: q = k = v = AdaRMSNorm(x), the already pinned Eq. 2."""
    rng = np.random.default_rng(3)
    R, D, Cd, Hd = 4, 24, 5, 6
    x = rng.standard_normal((R, D)).astype(np.float32)
    c = rng.standard_normal(Cd).astype(np.float32)
    W1, b1, W2, b2 = _mlp(rng, D, Cd, Hd)
    eye = np.eye(D, dtype=np.float32)
    q, k, v = orc.adarmsnorm_qkv(x, c, W1, b1, W2, b2, np.concatenate([eye, eye, eye]), 1, 1, D)
    y = orc.adarmsnorm(x, c, W1, b1, W2, b2)
    for o in (q, k, v):
        assert np.max(np.abs(o[:, 0, :] - y)) <= 1e-15


def test_packed_equals_three_separate_torch_linears():
    """The packed matrix gives what three separate projections give: torch.nn.functional.linear in fp64 on the norm output,
    head h of Q = rows [h d, (h+1) d) of W_Q (a transposed or mis-sliced weight fails here: Hq != Hkv, d != D)."""
    rng = np.random.default_rng(4)
    R, D, Cd, Hd, Hq, Hkv, d = 7, 40, 6, 9, 3, 2, 8
    x = (rng.standard_normal((R, D)) * 2).astype(np.float32)
    c = rng.standard_normal(Cd).astype(np.float32)
    W1, b1, W2, b2 = _mlp(rng, D, Cd, Hd)
    Wq = rng.standard_normal((Hq * d, D)).astype(np.float32); Wk = rng.standard_normal((Hkv * d, D)).astype(np.float32)
    Wv = rng.standard_normal((Hkv * d, D)).astype(np.float32)
    q, k, v = orc.adarmsnorm_qkv(x, c, W1, b1, W2, b2, np.concatenate([Wq, Wk, Wv]), Hq, Hkv, d)
    y = torch.from_numpy(orc.adarmsnorm(x, c, W1, b1, W2, b2))
    lin = lambda W: torch.nn.functional.linear(y, torch.from_numpy(W).double()).numpy()
    assert np.max(np.abs(q.reshape(R, -1) - lin(Wq))) <= 1e-12
    assert np.max(np.abs(k.reshape(R, -1) - lin(Wk))) <= 1e-12
    assert np.max(np.abs(v.reshape(R, -1) - lin(Wv))) <= 1e-12
    assert q.shape == (R, Hq, d) and k.shape == (R, Hkv, d) and v.shape == (R, Hkv, d)


def test_brute_force_and_row_scale_invariance():
    """Python loops over every term on a tiny case; and with eps = 0 the output does not change when a row of x is scaled
    (the norm divides the scale out), while it is linear in the weights."""
    rng = np.random.default_rng(5)
    R, D, Cd, Hd, Hq, Hkv, d = 2, 6, 2, 3, 2, 1, 2
    x = rng.standard_normal((R, D)).astype(np.float32)
    c = rng.standard_normal(Cd).astype(np.float32)
    W1, b1, W2, b2 = _mlp(rng, D, Cd, Hd)
    W = rng.standard_normal(((Hq + 2 * Hkv) * d, D)).astype(np.float32)
    q, k, v = orc.adarmsnorm_qkv(x, c, W1, b1, W2, b2, W, Hq, Hkv, d, eps=0.0)
    hid = [sum(float(W1[j, e]) * float(c[e]) for e in range(Cd)) + float(b1[j]) for j in range(Hd)]
    hid = [z / (1.0 + np.exp(-z)) for z in hid]
    gam = [1.0 + sum(float(W2[i, j]) * hid[j] for j in range(Hd)) + float(b2[i]) for i in range(D)]
    packed = np.concatenate([q.reshape(R, -1), k.reshape(R, -1), v.reshape(R, -1)], axis=1)
    for r in range(R):
        rms = np.sqrt(sum(float(x[r, i]) ** 2 for i in range(D)) / D)
        for n in range(W.shape[0]):
            want = sum(float(x[r, i]) / rms * gam[i] * float(W[n, i]) for i in range(D))
            assert abs(packed[r, n] - want) <= 1e-13
    q2, k2, v2 = orc.adarmsnorm_qkv(x * np.float32(4.0), c, W1, b1, W2, b2, W, Hq, Hkv, d, eps=0.0)
    assert np.max(np.abs(q2 - q)) <= 1e-13 and np.max(np.abs(v2 - v)) <= 1e-13
    q3, _, _ = orc.adarmsnorm_qkv(x, c, W1, b1, W2, b2, W * np.float32(2.0), Hq, Hkv, d, eps=0.0)
    assert np.max(np.abs(q3 - 2 * q)) <= 1e-13


# ---- adaptive norm + fused gate / up projections of a SwiGLU block (Sec. 3.3: "combine the Gate and Up projections") ----

def test_swiglu_hand_worked_example():
    """x = (3, 4), gate off, eps = 0: y = x / sqrt(12.5). Wg = [(1, 0)], Wu = [(0, 1)]: h = SiLU(y0) * y1."""
    x = np.array([[3.0, 4.0]], np.float32)
    z1 = np.zeros((1, 1), np.float32); zb = np.zeros(1, np.float32)
    h = orc.adarmsnorm_swiglu(x, np.zeros(1, np.float32), z1, zb, np.zeros((2, 1), np.float32), np.zeros(2, np.float32),
                              np.array([[1, 0]], np.float32), np.array([[0, 1]], np.float32), eps=0.0)
    r = np.sqrt(12.5)
    y0, y1 = 3 / r, 4 / r
    assert abs(h[0, 0] - y0 / (1 + np.exp(-y0)) * y1) <= 1e-15


def test_swiglu_matches_torch_fp64_and_is_not_symmetric():
    """h == silu(linear(y, Wg)) * linear(y, Wu) from torch in fp64; swapping Wg and Wu changes the result (the activation sits
    on the gate branch only), and a zero up-projection row gives exactly 0."""
    rng = np.random.default_rng(6)
    R, D, Cd, Hd, F = 5, 24, 4, 6, 10
    x = rng.standard_normal((R, D)).astype(np.float32)
    c = rng.standard_normal(Cd).astype(np.float32)
    W1, b1, W2, b2 = _mlp(rng, D, Cd, Hd)
    Wg = rng.standard_normal((F, D)).astype(np.float32) * np.float32(0.3)
    Wu = rng.standard_normal((F, D)).astype(np.float32) * np.float32(0.3)
    Wu[3] = 0
    h = orc.adarmsnorm_swiglu(x, c, W1, b1, W2, b2, Wg, Wu)
    y = torch.from_numpy(orc.adarmsnorm(x, c, W1, b1, W2, b2))
    Fn = torch.nn.functional
    want = (Fn.silu(Fn.linear(y, torch.from_numpy(Wg).double())) * Fn.linear(y, torch.from_numpy(Wu).double())).numpy()
    assert np.max(np.abs(h - want)) <= 1e-12
    assert np.all(h[:, 3] == 0.0)
    assert np.max(np.abs(orc.adarmsnorm_swiglu(x, c, W1, b1, W2, b2, Wu, Wg) - h)) > 1e-3


def test_swiglu_brute_force():
    rng = np.random.default_rng(7)
    R, D, Cd, Hd, F = 2, 5, 2, 3, 3
    x = rng.standard_normal((R, D)).astype(np.float32)
    c = rng.standard_normal(Cd).astype(np.float32)
    W1, b1, W2, b2 = _mlp(rng, D, Cd, Hd)
    Wg = rng.standard_normal((F, D)).astype(np.float32); Wu = rng.standard_normal((F, D)).astype(np.float32)
    h = orc.adarmsnorm_swiglu(x, c, W1, b1, W2, b2, Wg, Wu, eps=1e-5)
    hid = [sum(float(W1[j, e]) * float(c[e]) for e in range(Cd)) + float(b1[j]) for j in range(Hd)]
    hid = [z / (1.0 + np.exp(-z)) for z in hid]
    gam = [1.0 + sum(float(W2[i, j]) * hid[j] for j in range(Hd)) + float(b2[i]) for i in range(D)]
    for r in range(R):
        rms = np.sqrt(sum(float(x[r, i]) ** 2 for i in range(D)) / D + 1e-5)
        y = [float(x[r, i]) / rms * gam[i] for i in range(D)]
        for f in range(F):
            g = sum(y[i] * float(Wg[f, i]) for i in range(D)); u = sum(y[i] * float(Wu[f, i]) for i in range(D))
            assert abs(h[r, f] - g / (1.0 + np.exp(-g)) * u) <= 1e-13
