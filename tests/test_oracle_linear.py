"""Pins for the oracle's plain projection with residual (the attention output projection and the SwiGLU down projection of
the action expert, Sec. 3.3): out = res + a W^T with W holding one row per output feature."""
import numpy as np
import torch

from oracle import reflex_oracle as orc


def test_hand_worked_example():
    """a = (1, 2, 3), W rows (1, 0, -1) and (2, 1, 0), res = (10, 20): out = (10 + 1 - 3, 20 + 2 + 2) = (8, 24)."""
    a = np.array([[1.0, 2.0, 3.0]], np.float32)
    W = np.array([[1, 0, -1], [2, 1, 0]], np.float32)
    out = orc.linear_residual(a, W, np.array([[10.0, 20.0]], np.float32))
    assert np.array_equal(out, [[8.0, 24.0]])
    assert np.array_equal(orc.linear_residual(a, W), [[-2.0, 4.0]])          # no residual


def test_equals_torch_linear_plus_residual_fp64():
    """Non-square shapes (M, K, N all different): a transposed weight matrix, a residual indexed by the wrong axis or a
    dropped residual fails."""
    rng = np.random.default_rng(11)
    M, K, N = 7, 19, 5
    a = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    res = rng.standard_normal((M, N)).astype(np.float32)
    want = (torch.nn.functional.linear(torch.from_numpy(a).double(), torch.from_numpy(W).double()) + torch.from_numpy(res).double()).numpy()
    assert np.max(np.abs(orc.linear_residual(a, W, res) - want)) <= 1e-13
    assert np.max(np.abs(orc.linear_residual(a, W) - (want - res))) <= 1e-13


def test_brute_force_python_loops():
    rng = np.random.default_rng(12)
    M, K, N = 3, 4, 6
    a = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    res = rng.standard_normal((M, N)).astype(np.float32)
    out = orc.linear_residual(a, W, res)
    for r in range(M):
        for n in range(N):
            acc = float(res[r, n])
            for i in range(K):
                acc += float(a[r, i]) * float(W[n, i])
            assert abs(out[r, n] - acc) <= 1e-14


def test_identity_weights_and_linearity():
    """W = I returns a + res; the map is linear in a and in W; a zero W returns the residual bit for bit."""
    rng = np.random.default_rng(13)
    M, K = 5, 8
    a = rng.standard_normal((M, K)).astype(np.float32)
    res = rng.standard_normal((M, K)).astype(np.float32)
    assert np.array_equal(orc.linear_residual(a, np.eye(K, dtype=np.float32), res), a.astype(np.float64) + res)
    W = rng.standard_normal((3, K)).astype(np.float32)
    W2 = rng.standard_normal((3, K)).astype(np.float32)
    lhs = orc.linear_residual(a, W) + orc.linear_residual(a, W2)
    assert np.max(np.abs(lhs - a.astype(np.float64) @ (W.astype(np.float64) + W2).T)) <= 1e-13
    r3 = rng.standard_normal((M, 3)).astype(np.float32)
    assert np.array_equal(orc.linear_residual(a, np.zeros((3, K), np.float32), r3), r3.astype(np.float64))


def test_expert_oracle_uses_the_same_projection():
    """The whole-step oracle's residual updates are this function (numpy products there): both agree on random data."""
    rng = np.random.default_rng(14)
    h = rng.standard_normal((6, 10))
    o = rng.standard_normal((6, 12)).astype(np.float32)
    Wo = rng.standard_normal((10, 12)).astype(np.float32)
    want = h + o.astype(np.float64) @ Wo.astype(np.float64).T
    got = orc.linear_residual(o, Wo, h.astype(np.float32))
    assert np.max(np.abs(got - want)) <= 1e-6          # (h passes through float32 on its way into the C routine)
