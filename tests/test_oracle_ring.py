"""Pins for the sliding ring (Sec. 3.1 FIFO of size N; Sec. 3.4 / App. B.2 circular write pointer;
App. B.1 "returns eviction count") and for timestep invariance of the cached regions."""
import collections

import numpy as np
import pytest

from oracle import reflex_oracle as orc


def _tok(L, m, Hkv, d, first_id):
    """Tokens whose every element equals their global append index: content identifies the token."""
    k = np.empty((L, m, Hkv, d), np.float32)
    for i in range(m):
        k[:, i] = float(first_id + i)
    return k, -k


@pytest.mark.parametrize("N,head0,seed", [(1, 0, 0), (2, 1, 1), (5, 3, 2), (7, 0, 3), (16, 9, 4)])
def test_ring_matches_deque_on_random_trace(N, head0, seed):
    rng = np.random.default_rng(seed)
    L, Hkv, d = 2, 1, 2
    c = orc.OracleCache(L, 1, Hkv, d, 1, N, head0=[head0])
    dq = collections.deque(maxlen=N)
    g = 0
    for _ in range(60):
        m = int(rng.integers(1, N + 1))
        before = len(dq)
        k, v = _tok(L, m, Hkv, d, g)
        ev = c.append_sliding(0, k, v)
        for i in range(m):
            dq.append(g + i)
        g += m
        assert ev == before + m - len(dq)                      # tokens that fell out of the FIFO
        assert c.count[0] == len(dq) and c.total[0] == g
        assert c.head[0] == (head0 + g) % N                    # write pointer geometry
        sm = c.slot_map(0)
        ids = [int(c.k_ring[0, 0, s, 0, 0]) for s in sm[: c.count[0]]]
        assert ids == list(dq)                                 # FIFO order, oldest first
        assert all(s == -1 for s in sm[c.count[0]:])
        for layer in range(L):                                 # every layer holds the same tokens
            assert [int(c.k_ring[layer, 0, s, 0, 0]) for s in sm[: c.count[0]]] == list(dq)
            assert [int(-c.v_ring[layer, 0, s, 0, 0]) for s in sm[: c.count[0]]] == list(dq)


def test_cfg1_closed_form_trace():
    """Tiny config: N = 16, one token per tick, 40 ticks from head 0."""
    N = 16
    c = orc.OracleCache(1, 1, 1, 2, 1, N)
    evicted_total = 0
    for n in range(1, 41):
        k, v = _tok(1, 1, 1, 2, n)
        evicted_total += c.append_sliding(0, k, v)
        assert c.head[0] == n % 16
        assert c.count[0] == min(n, 16)
        assert evicted_total == max(0, n - 16)
        survivors = [int(c.k_ring[0, 0, s, 0, 0]) for s in c.slot_map(0)[: c.count[0]]]
        assert survivors == list(range(max(1, n - 15), n + 1))
    assert evicted_total == 24


def test_slot_of_global_index_and_period():
    N, head0 = 6, 4
    c = orc.OracleCache(1, 1, 1, 1, 1, N, head0=[head0])
    for g in range(3 * N):
        k, v = _tok(1, 1, 1, 1, g)
        c.append_sliding(0, k, v)
        assert int(c.k_ring[0, 0, (head0 + g) % N, 0, 0]) == g
        if (g + 1) % N == 0:
            assert c.head[0] == head0                          # N single appends return the pointer


def test_m_bounds_and_multi_token_append():
    c = orc.OracleCache(1, 1, 1, 1, 1, 4)
    with pytest.raises(ValueError):
        c.append_sliding(0, np.zeros((1, 0, 1, 1), np.float32), np.zeros((1, 0, 1, 1), np.float32))
    with pytest.raises(ValueError):
        c.append_sliding(0, np.zeros((1, 5, 1, 1), np.float32), np.zeros((1, 5, 1, 1), np.float32))
    k, v = _tok(1, 3, 1, 1, 0); assert c.append_sliding(0, k, v) == 0
    k, v = _tok(1, 4, 1, 1, 3); assert c.append_sliding(0, k, v) == 3          # m = N replaces everything
    assert [int(c.k_ring[0, 0, s, 0, 0]) for s in c.slot_map(0)] == [3, 4, 5, 6]


def test_streams_are_independent_and_static_untouched_by_appends():
    rng = np.random.default_rng(0)
    c = orc.OracleCache(2, 3, 1, 4, 5, 3, head0=[0, 1, 2])
    for b in range(3):
        c.init_static(b, rng.standard_normal((2, 5, 1, 4)).astype(np.float32), rng.standard_normal((2, 5, 1, 4)).astype(np.float32))
    snap_static = c.k_static.copy()
    snap_ring = c.k_ring.copy()
    k, v = _tok(2, 2, 1, 4, 100)
    c.append_sliding(1, k, v)
    assert np.array_equal(c.k_static, snap_static)
    assert np.array_equal(c.k_ring[:, 0], snap_ring[:, 0]) and np.array_equal(c.k_ring[:, 2], snap_ring[:, 2])
    assert c.head == [0, 0, 2] and c.count == [0, 2, 0]


def test_shorter_new_prefix_masks_stale_tail_and_keeps_ring():
    """A new observation with a shorter prefix: static_len alone decides validity; the ring is not reset."""
    rng = np.random.default_rng(1)
    c = orc.OracleCache(1, 1, 1, 4, 6, 3)
    c.init_static(0, rng.standard_normal((1, 6, 1, 4)).astype(np.float32), rng.standard_normal((1, 6, 1, 4)).astype(np.float32))
    k, v = _tok(1, 2, 1, 4, 0); c.append_sliding(0, k, v)
    ks = rng.standard_normal((1, 4, 1, 4)).astype(np.float32); vs = rng.standard_normal((1, 4, 1, 4)).astype(np.float32)
    c.init_static(0, ks, vs)
    assert c.static_len[0] == 4 and c.count[0] == 2
    c.k_static[0, 0, 4:] = np.nan; c.v_static[0, 0, 4:] = np.nan      # stale tail must never be read
    q = rng.standard_normal((2, 2, 4)).astype(np.float32); kd = rng.standard_normal((2, 1, 4)).astype(np.float32)
    vd = rng.standard_normal((2, 1, 4)).astype(np.float32)
    for part in (False, True):
        assert np.isfinite(c.attention(0, 0, q, kd, vd, partitioned=part)).all()


def test_cached_regions_do_not_change_across_denoising_steps():
    """Timestep invariance (Sec. 3.1): attention at any step reads, never writes, prefix and ring."""
    rng = np.random.default_rng(2)
    c = orc.OracleCache(1, 1, 1, 8, 4, 3)
    c.init_static(0, rng.standard_normal((1, 4, 1, 8)).astype(np.float32), rng.standard_normal((1, 4, 1, 8)).astype(np.float32))
    k, v = _tok(1, 2, 1, 8, 0); c.append_sliding(0, k, v)
    snap = [a.tobytes() for a in (c.k_static, c.v_static, c.k_ring, c.v_ring)]
    state = (list(c.head), list(c.count), list(c.static_len))
    for step in range(4):
        q = rng.standard_normal((3, 2, 8)).astype(np.float32); kd = rng.standard_normal((3, 1, 8)).astype(np.float32)
        vd = rng.standard_normal((3, 1, 8)).astype(np.float32)
        c.attention(0, 0, q, kd, vd); c.attention(0, 0, q, kd, vd, partitioned=True)
        assert [a.tobytes() for a in (c.k_static, c.v_static, c.k_ring, c.v_ring)] == snap
        assert (list(c.head), list(c.count), list(c.static_len)) == state
