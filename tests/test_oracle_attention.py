"""Pins for the oracle's attention (Eq. 1, Proposition 1). Each check is independent of the
oracle's own code path: a library routine, a closed form, an invariant or a special case."""
import numpy as np
import pytest
import torch

from oracle import reflex_oracle as orc


def _rand_cache(rng, L=1, B=1, Hkv=1, d=8, S_max=6, N=5, S=None, appends=0, head0=0):
    c = orc.OracleCache(L, B, Hkv, d, S_max, N, head0=[head0] * B)
    S = S_max if S is None else S
    for b in range(B):
        c.init_static(b, rng.standard_normal((L, S, Hkv, d)).astype(np.float32),
                      rng.standard_normal((L, S, Hkv, d)).astype(np.float32))
        for _ in range(appends):
            c.append_sliding(b, rng.standard_normal((L, 1, Hkv, d)).astype(np.float32),
                             rng.standard_normal((L, 1, Hkv, d)).astype(np.float32))
    return c


def _numpy_attention(q, kc, vc, G, scale, mask=None):
    """softmax(Q K^T * scale) V in numpy fp64, KV heads repeated for GQA."""
    q = q.astype(np.float64); kc = np.repeat(kc.astype(np.float64), G, axis=1); vc = np.repeat(vc.astype(np.float64), G, axis=1)
    s = np.einsum("ihe,jhe->hij", q, kc) * scale
    if mask is not None:
        s = np.where(mask[None], s, -np.inf)
    s = s - s.max(-1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(-1, keepdims=True)
    return np.einsum("hij,jhe->ihe", p, vc)


CASES = [
    # (Hq, Hkv, d, S_max, S, N, appends, head0, T)
    (2, 1, 8, 6, 6, 5, 0, 0, 3),     # empty ring
    (2, 1, 8, 6, 6, 5, 3, 0, 3),     # count < N
    (4, 2, 16, 7, 4, 5, 5, 3, 4),    # exactly full, wrapped, S < S_max
    (4, 2, 16, 7, 0, 5, 12, 2, 4),   # S = 0, wrapped more than twice
    (8, 1, 32, 9, 9, 4, 9, 1, 5),    # GQA 8:1
    (3, 3, 4, 2, 2, 1, 2, 0, 1),     # N = 1, T = 1, MHA
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("dyn_mask", [0, 1])
def test_partitioned_equals_definition(case, dyn_mask):
    """Proposition 1: region-wise evaluation in physical ring order == attention over the concatenation."""
    Hq, Hkv, d, S_max, S, N, appends, head0, T = case
    rng = np.random.default_rng(hash(case) % 2**32)
    c = _rand_cache(rng, 2, 2, Hkv, d, S_max, N, S, appends, head0)
    for b in range(2):
        for layer in range(2):
            q = rng.standard_normal((T, Hq, d)).astype(np.float32)
            kd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
            vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
            a = c.attention(b, layer, q, kd, vd, dyn_mask)
            p = c.attention(b, layer, q, kd, vd, dyn_mask, partitioned=True)
            assert np.max(np.abs(a - p)) <= 1e-12


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("dyn_mask", [0, 1])
def test_against_numpy_and_torch_sdpa(case, dyn_mask):
    """Both oracle forms == numpy fp64 softmax(QK^T/sqrt d)V and == torch SDPA (fp64, CPU) on the
    hand-built concatenation [static[:S]; ring oldest->newest; dynamic]."""
    Hq, Hkv, d, S_max, S, N, appends, head0, T = case
    rng = np.random.default_rng(1 + hash(case) % 2**32)
    L = 1
    c = orc.OracleCache(L, 1, Hkv, d, S_max, N, head0=[head0])
    ks = rng.standard_normal((L, S, Hkv, d)).astype(np.float32); vs = rng.standard_normal((L, S, Hkv, d)).astype(np.float32)
    c.init_static(0, ks, vs)
    hist_k, hist_v = [], []
    for _ in range(appends):
        kn = rng.standard_normal((L, 1, Hkv, d)).astype(np.float32); vn = rng.standard_normal((L, 1, Hkv, d)).astype(np.float32)
        c.append_sliding(0, kn, vn)
        hist_k.append(kn[0, 0]); hist_v.append(vn[0, 0])
    # FIFO of size N, written out independently of the oracle's slot arithmetic: keep the last N appends
    hist_k, hist_v = hist_k[-N:], hist_v[-N:]
    q = rng.standard_normal((T, Hq, d)).astype(np.float32)
    kd = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    kc = np.concatenate([ks[0]] + ([np.stack(hist_k)] if hist_k else []) + [kd])
    vc = np.concatenate([vs[0]] + ([np.stack(hist_v)] if hist_v else []) + [vd])
    n_prefix = kc.shape[0] - T
    mask = np.ones((T, kc.shape[0]), bool)
    if dyn_mask:
        for i in range(T):
            mask[i, n_prefix + i + 1:] = False
    scale = 1.0 / np.sqrt(d)
    ref = _numpy_attention(q, kc, vc, Hq // Hkv, scale, mask)
    tq = torch.from_numpy(q).double().permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.repeat(kc, Hq // Hkv, axis=1)).double().permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(vc, Hq // Hkv, axis=1)).double().permute(1, 0, 2)[None]
    sd = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask))[0].permute(1, 0, 2).numpy()
    for part in (False, True):
        got = c.attention(0, 0, q, kd, vd, dyn_mask, partitioned=part)
        assert np.max(np.abs(got - ref)) <= 1e-12
        assert np.max(np.abs(got - sd)) <= 1e-10


def test_zero_query_gives_mean_of_valid_values():
    """q = 0 -> uniform weights -> output is the mean of exactly the valid V rows. Empty ring slots
    and the stale tail of a shortened prefix are poisoned with NaN: any leak shows."""
    rng = np.random.default_rng(3)
    Hq, Hkv, d, S_max, N, T = 4, 2, 8, 10, 6, 3
    c = orc.OracleCache(1, 1, Hkv, d, S_max, N, head0=[4])
    c.k_static[:] = np.nan; c.v_static[:] = np.nan; c.k_ring[:] = np.nan; c.v_ring[:] = np.nan
    S = 7
    ks = rng.standard_normal((1, S, Hkv, d)).astype(np.float32); vs = rng.standard_normal((1, S, Hkv, d)).astype(np.float32)
    c.init_static(0, ks, vs)
    app_v = []
    for _ in range(4):  # count = 4 < N, wraps (head0 = 4)
        kn = rng.standard_normal((1, 1, Hkv, d)).astype(np.float32); vn = rng.standard_normal((1, 1, Hkv, d)).astype(np.float32)
        c.append_sliding(0, kn, vn); app_v.append(vn[0, 0])
    kd = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    q = np.zeros((T, Hq, d), np.float32)
    allv = np.concatenate([vs[0], np.stack(app_v), vd]).astype(np.float64)  # [n][Hkv][d]
    want = allv.mean(0)  # [Hkv][d]
    for part in (False, True):
        got = c.attention(0, 0, q, kd, vd, 0, partitioned=part)
        assert np.isfinite(got).all()
        for h in range(Hq):
            assert np.max(np.abs(got[:, h] - want[h // 2][None])) <= 1e-13
    # causal: query i sees prefix + ring + dynamic 0..i
    for part in (False, True):
        got = c.attention(0, 0, q, kd, vd, 1, partitioned=part)
        for i in range(T):
            want_i = np.concatenate([vs[0], np.stack(app_v), vd[: i + 1]]).astype(np.float64).mean(0)
            for h in range(Hq):
                assert np.max(np.abs(got[i, h] - want_i[h // 2])) <= 1e-13


def test_dominant_key_and_key_shift_invariance():
    rng = np.random.default_rng(4)
    Hq, Hkv, d, S_max, N, T = 2, 1, 16, 5, 4, 3
    for region in ("static", "ring", "dyn"):
        c = _rand_cache(rng, 1, 1, Hkv, d, S_max, N, S_max, 6, 1)
        q = rng.standard_normal((T, Hq, d)).astype(np.float32)
        kd = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
        # put a key with a huge logit for query (0, head 0) into one region
        big = (q[0, 0] * 400.0).astype(np.float32)
        if region == "static":
            c.k_static[0, 0, 2, 0] = big; target = c.v_static[0, 0, 2, 0]
        elif region == "ring":
            c.k_ring[0, 0, 3, 0] = big; target = c.v_ring[0, 0, 3, 0]
        else:
            kd[1, 0] = big; target = vd[1, 0]
        for part in (False, True):
            got = c.attention(0, 0, q, kd, vd, 0, partitioned=part)
            assert np.max(np.abs(got[0, 0] - target.astype(np.float64))) <= 1e-12
    # adding the same vector u to every key shifts each query's logits by a constant: output unchanged
    c = _rand_cache(rng, 1, 1, Hkv, d, S_max, N, 3, 6, 2)
    q = rng.standard_normal((T, Hq, d)).astype(np.float32)
    kd = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    base = c.attention(0, 0, q, kd, vd, 0)
    u = rng.integers(-2, 3, size=(d,)).astype(np.float32) * 0.5  # exactly representable shifts
    c.k_static = (c.k_static + u).astype(np.float32); c.k_ring = (c.k_ring + u).astype(np.float32)
    for part in (False, True):
        got = c.attention(0, 0, q, (kd + u).astype(np.float32), vd, 0, partitioned=part)
        assert np.max(np.abs(got - base)) <= 1e-5  # keys move by fp32 rounding of k+u only


def test_permutation_invariance_of_ring_and_static():
    rng = np.random.default_rng(5)
    Hq, Hkv, d, S_max, N, T = 4, 2, 8, 6, 5, 3
    c = _rand_cache(rng, 1, 1, Hkv, d, S_max, N, S_max, 9, 2)
    q = rng.standard_normal((T, Hq, d)).astype(np.float32)
    kd = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    base = c.attention(0, 0, q, kd, vd, 0)
    pr = rng.permutation(N); ps = rng.permutation(S_max)
    c.k_ring = c.k_ring[:, :, pr].copy(); c.v_ring = c.v_ring[:, :, pr].copy()
    c.k_static = c.k_static[:, :, ps].copy(); c.v_static = c.v_static[:, :, ps].copy()
    for part in (False, True):
        assert np.max(np.abs(c.attention(0, 0, q, kd, vd, 0, partitioned=part) - base)) <= 1e-12


def test_causal_first_query_equals_single_dynamic_token():
    rng = np.random.default_rng(6)
    Hq, Hkv, d, S_max, N, T = 2, 1, 8, 4, 3, 5
    c = _rand_cache(rng, 1, 1, Hkv, d, S_max, N, S_max, 2, 0)
    q = rng.standard_normal((T, Hq, d)).astype(np.float32)
    kd = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    for part in (False, True):
        causal = c.attention(0, 0, q, kd, vd, 1, partitioned=part)
        single = c.attention(0, 0, q[:1], kd[:1], vd[:1], 0, partitioned=part)
        assert np.max(np.abs(causal[0] - single[0])) <= 1e-13
        full_last = c.attention(0, 0, q, kd, vd, 0, partitioned=part)
        assert np.max(np.abs(causal[-1] - full_last[-1])) <= 1e-13  # last query sees everything either way


def test_uninitialised_prefix_is_an_error_and_scale_override():
    c = orc.OracleCache(1, 1, 1, 4, 2, 2)
    z = np.zeros((1, 1, 4), np.float32)
    with pytest.raises(RuntimeError):
        c.attention(0, 0, z, z, z)
    rng = np.random.default_rng(7)
    c = _rand_cache(rng, 1, 1, 1, 4, 2, 2, 2, 1, 0)
    q = rng.standard_normal((2, 1, 4)).astype(np.float32); kd = rng.standard_normal((2, 1, 4)).astype(np.float32)
    vd = rng.standard_normal((2, 1, 4)).astype(np.float32)
    a = c.attention(0, 0, q, kd, vd, 0, scale=0.25)
    b = c.attention(0, 0, (q * 0.5).astype(np.float32), kd, vd, 0, scale=0.5)  # scaling q by 1/2 == halving scale
    assert np.max(np.abs(a - b)) <= 1e-13


def test_stale_dynamic_kv_is_wrong():
    """Negative control (Sec. 4.4, cache ablation): reusing step-0 dynamic K/V at a later step, i.e. a
    cache that ignores the timestep, gives a visibly different answer."""
    rng = np.random.default_rng(8)
    Hq, Hkv, d, S_max, N, T = 2, 1, 16, 8, 4, 6
    c = _rand_cache(rng, 1, 1, Hkv, d, S_max, N, S_max, 4, 0)
    q = rng.standard_normal((T, Hq, d)).astype(np.float32)
    kd0 = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd0 = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    kd1 = rng.standard_normal((T, Hkv, d)).astype(np.float32); vd1 = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    right = c.attention(0, 0, q, kd1, vd1, 0)
    stale = c.attention(0, 0, q, kd0, vd0, 0)
    assert np.mean((right - stale) ** 2) > 1e-2
