"""CPU oracle for the Reflex action-expert hot path: Python front of reflex_oracle.c.

TEST INFRASTRUCTURE ONLY. Only tests, the smoke check and the bench's CPU-baseline leg may import
this module; the product (the CUDA library and its binding) never does, and this module imports
nothing from the product. It is slow and plain on purpose.

What lives here (everything else is in reflex_oracle.c):
  * the cache state of Sec. 3.1 -- pinned static prefix, sliding FIFO ring, per stream -- and the
    O(1) circular-pointer append of Sec. 3.4 / Appendix B.2 (integer arithmetic, exact);
  * the gather of the logical context [pinned ; sliding in FIFO order ; dynamic] that the
    by-definition attention (Eq. 1) consumes.

Pins (tests/test_oracle_*.py): numpy/torch fp64 library attention, closed forms (zero query ->
mean of valid V; dominant key; key-shift invariance), permutation invariance, causal special case,
collections.deque for the ring, torch rms_norm and hand-computed gates for AdaRMSNorm, closed-form
Euler trajectories. The paper's own numeric tables need trained weights and simulators, so no
printed value pins this oracle: parity against the paper's tables is unpinned by construction.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "reflex_oracle.c")
_LIB = os.path.join(_HERE, "libreflex_oracle.so")


def build(force: bool = False) -> str:
    """Compile reflex_oracle.c with gcc (OpenMP). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        i, d = ctypes.c_int, ctypes.c_double
        _lib.reflex_oracle_attention_def.argtypes = [fp, fp, fp, i, i, i, i, i, i, i, d, dp]
        _lib.reflex_oracle_attention_def.restype = i
        _lib.reflex_oracle_attention_part.argtypes = [fp, fp, fp, i, fp, fp, i, i, i, fp, fp, i, i, i, i, i, d, dp]
        _lib.reflex_oracle_attention_part.restype = i
        _lib.reflex_oracle_adarmsnorm.argtypes = [fp, fp, fp, fp, fp, fp, i, i, i, i, d, dp, dp]
        _lib.reflex_oracle_adarmsnorm.restype = i
        _lib.reflex_oracle_adarmsnorm_linear.argtypes = [fp, dp, fp, i, i, i, d, dp]
        _lib.reflex_oracle_adarmsnorm_linear.restype = i
        _lib.reflex_oracle_adarmsnorm_swiglu.argtypes = [fp, dp, fp, fp, i, i, i, d, dp]
        _lib.reflex_oracle_adarmsnorm_swiglu.restype = i
        _lib.reflex_oracle_linear_residual.argtypes = [fp, fp, fp, i, i, i, dp]
        _lib.reflex_oracle_linear_residual.restype = i
        _lib.reflex_oracle_flow_step.argtypes = [dp, fp, ctypes.c_long, i]
        _lib.reflex_oracle_flow_step.restype = None
        _lib.reflex_oracle_flow_time.argtypes = [i, i]
        _lib.reflex_oracle_flow_time.restype = d
        _lib.reflex_oracle_max_threads.restype = i
    return _lib


def max_threads() -> int:
    return int(lib().reflex_oracle_max_threads())


def _f(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _dptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


# ------------------------------------------------------------------------------------------------
# stateless pieces
# ------------------------------------------------------------------------------------------------

def attention_def(q, kctx, vctx, n_prefix, dyn_mask=0, scale=None):
    """Eq. 1 by definition over an explicit context. q [T][Hq][d], kctx/vctx [n][Hkv][d] -> [T][Hq][d] f64."""
    q, qp = _f(q); kctx, kp = _f(kctx); vctx, vp = _f(vctx)
    T, Hq, d = q.shape
    n, Hkv, _ = kctx.shape
    scale = 1.0 / np.sqrt(float(d)) if scale is None else float(scale)
    out = np.empty((T, Hq, d), np.float64)
    rc = lib().reflex_oracle_attention_def(qp, kp, vp, T, Hq, Hkv, d, n, int(n_prefix), int(dyn_mask), scale, _dptr(out))
    if rc != 0:
        raise MemoryError("oracle attention_def")
    return out


def attention_part(q, k_s, v_s, S, k_r, v_r, head, count, k_d, v_d, dyn_mask=0, scale=None):
    """Eq. 1 region by region with the (m, l, acc) merge; ring passed in physical slot order."""
    q, qp = _f(q); k_s, ksp = _f(k_s); v_s, vsp = _f(v_s); k_r, krp = _f(k_r); v_r, vrp = _f(v_r)
    k_d, kdp = _f(k_d); v_d, vdp = _f(v_d)
    T, Hq, d = q.shape
    Hkv = k_d.shape[1]
    N = k_r.shape[0]
    scale = 1.0 / np.sqrt(float(d)) if scale is None else float(scale)
    out = np.empty((T, Hq, d), np.float64)
    rc = lib().reflex_oracle_attention_part(qp, ksp, vsp, int(S), krp, vrp, N, int(head), int(count), kdp, vdp,
                                            T, Hq, Hkv, d, int(dyn_mask), scale, _dptr(out))
    if rc != 0:
        raise MemoryError("oracle attention_part")
    return out


def adarmsnorm(x, c, W1, b1, W2, b2, eps=1e-6, return_gate=False):
    """Eq. 2 for one stream: x [R][D], c [Cd] -> y [R][D] f64 (and gamma [D])."""
    x, xp = _f(x); c, cp = _f(c); W1, w1p = _f(W1); b1, b1p = _f(b1); W2, w2p = _f(W2); b2, b2p = _f(b2)
    R, D = x.shape
    Hd, Cd = W1.shape
    y = np.empty((R, D), np.float64)
    g = np.empty((D,), np.float64)
    rc = lib().reflex_oracle_adarmsnorm(xp, cp, w1p, b1p, w2p, b2p, R, D, Cd, Hd, float(eps), _dptr(y), _dptr(g))
    if rc != 0:
        raise MemoryError("oracle adarmsnorm")
    return (y, g) if return_gate else y


def adarmsnorm_batched(x, cond, W1, b1, W2, b2, eps=1e-6):
    """x [B][R][D], cond [B][Cd]: one gate per stream."""
    return np.stack([adarmsnorm(x[b], cond[b], W1, b1, W2, b2, eps) for b in range(x.shape[0])])


def adarmsnorm_qkv(x, c, W1, b1, W2, b2, Wqkv, Hq, Hkv, d, eps=1e-6):
    """Eq. 2 followed by the packed projection W_QKV = [W_Q; W_K; W_V] for one stream:
    x [R][D], Wqkv [(Hq + 2 Hkv) d][D] -> q [R][Hq][d], k [R][Hkv][d], v [R][Hkv][d], all f64."""
    _, g = adarmsnorm(x, c, W1, b1, W2, b2, eps, return_gate=True)
    x, xp = _f(x); Wqkv, wp = _f(Wqkv)
    R, D = x.shape
    Nout = Wqkv.shape[0]
    assert Nout == (Hq + 2 * Hkv) * d and Wqkv.shape[1] == D
    out = np.empty((R, Nout), np.float64)
    rc = lib().reflex_oracle_adarmsnorm_linear(xp, _dptr(g), wp, R, D, Nout, float(eps), _dptr(out))
    if rc != 0:
        raise MemoryError("oracle adarmsnorm_linear")
    nq, nk = Hq * d, Hkv * d
    return out[:, :nq].reshape(R, Hq, d), out[:, nq:nq + nk].reshape(R, Hkv, d), out[:, nq + nk:].reshape(R, Hkv, d)


def adarmsnorm_swiglu(x, c, W1, b1, W2, b2, Wg, Wu, eps=1e-6):
    """Eq. 2 followed by the fused gate / up projections of a SwiGLU block for one stream:
    x [R][D], Wg, Wu [F][D] -> h = SiLU(y Wg^T) * (y Wu^T), [R][F] f64."""
    _, g = adarmsnorm(x, c, W1, b1, W2, b2, eps, return_gate=True)
    x, xp = _f(x); Wg, gp = _f(Wg); Wu, up = _f(Wu)
    R, D = x.shape
    F = Wg.shape[0]
    assert Wg.shape == (F, D) and Wu.shape == (F, D)
    h = np.empty((R, F), np.float64)
    rc = lib().reflex_oracle_adarmsnorm_swiglu(xp, _dptr(g), gp, up, R, D, F, float(eps), _dptr(h))
    if rc != 0:
        raise MemoryError("oracle adarmsnorm_swiglu")
    return h


def linear_residual(a, W, res=None):
    """A plain projection with its residual: a [M][K], W [N][K], res [M][N] or None -> res + a W^T, [M][N] f64."""
    a, ap = _f(a); W, wp = _f(W)
    M, K = a.shape
    N = W.shape[0]
    assert W.shape == (N, K)
    rp = None
    if res is not None:
        res, rp = _f(res)
        assert res.shape == (M, N)
    out = np.empty((M, N), np.float64)
    rc = lib().reflex_oracle_linear_residual(ap, wp, rp, M, K, N, _dptr(out))
    if rc != 0:
        raise MemoryError("oracle linear_residual")
    return out


def flow_step(x, v, K):
    """In-place Euler update of a float64 array x with velocity v: x += (-1/K) v."""
    assert x.dtype == np.float64 and x.flags.c_contiguous
    v, vp = _f(v)
    assert v.size == x.size
    lib().reflex_oracle_flow_step(_dptr(x), vp, x.size, int(K))
    return x


def flow_time(k, K):
    return float(lib().reflex_oracle_flow_time(int(k), int(K)))


# ------------------------------------------------------------------------------------------------
# cache state: pinned prefix + sliding FIFO ring (Sec. 3.1, Sec. 3.4, Appendix B.1/B.2)
# ------------------------------------------------------------------------------------------------

class OracleCache:
    """Per-stream partitioned KV cache. Arrays are fp32 holding storage-dtype values.

    static: [L][B][S_max][Hkv][d]   ring: [L][B][N][Hkv][d] in physical slot order.
    head[b]  = next write slot (the write pointer of Appendix B.2), count[b] = live ring tokens,
    total[b] = tokens ever appended, static_len[b] = valid prefix rows (-1 = never initialised).
    """

    def __init__(self, L, B, Hkv, d, S_max, N, head0=None):
        self.L, self.B, self.Hkv, self.d, self.S_max, self.N = L, B, Hkv, d, S_max, N
        self.k_static = np.zeros((L, B, S_max, Hkv, d), np.float32)
        self.v_static = np.zeros_like(self.k_static)
        self.k_ring = np.zeros((L, B, N, Hkv, d), np.float32)
        self.v_ring = np.zeros_like(self.k_ring)
        self.static_len = [-1] * B
        self.head = [0] * B if head0 is None else [int(h) % N for h in head0]
        self.count = [0] * B
        self.total = [0] * B

    # Sec. 3.1: the static prefix is computed once per observation and pinned.
    def init_static(self, b, k_s, v_s):
        """k_s, v_s [L][S][Hkv][d]; rows [0,S) are overwritten, nothing else is touched."""
        S = k_s.shape[1]
        if not (0 <= S <= self.S_max):
            raise ValueError("S out of range")
        self.k_static[:, b, :S] = k_s
        self.v_static[:, b, :S] = v_s
        self.static_len[b] = S

    # Sec. 3.4 "Asynchronous Pipeline": the producer hands over a new prefix while the consumer still reads the current one.
    # By definition: staging changes nothing that attention sees; committing replaces the prefix as a whole.
    def stage_static(self, b, k_s, v_s):
        if not (0 <= k_s.shape[1] <= self.S_max):
            raise ValueError("S out of range")
        if not hasattr(self, "_staged"):
            self._staged = {}
        self._staged[b] = (np.array(k_s, np.float32), np.array(v_s, np.float32))

    def commit_static(self, b):
        k_s, v_s = self._staged.pop(b)
        S = k_s.shape[1]
        self.k_static[:, b] = np.nan            # the previous prefix is gone entirely (a read of stale rows shows up)
        self.v_static[:, b] = np.nan
        self.k_static[:, b, :S] = k_s
        self.v_static[:, b, :S] = v_s
        self.static_len[b] = S

    # Sec. 3.4 / App. B.1-B.2: circular write pointer, FIFO eviction of the oldest tokens, in all layers.
    def append_sliding(self, b, k_n, v_n):
        """k_n, v_n [L][m][Hkv][d]. Returns the number of tokens evicted."""
        m = k_n.shape[1]
        if not (1 <= m <= self.N):
            raise ValueError("m out of range")
        evicted = max(0, self.count[b] + m - self.N)
        for i in range(m):
            slot = (self.head[b] + i) % self.N
            self.k_ring[:, b, slot] = k_n[:, i]
            self.v_ring[:, b, slot] = v_n[:, i]
        self.head[b] = (self.head[b] + m) % self.N
        self.count[b] = min(self.count[b] + m, self.N)
        self.total[b] += m
        return evicted

    def slot_map(self, b):
        """slot_of_age [N]: physical slot of the token of age j (0 = oldest), -1 beyond count."""
        out = [-1] * self.N
        for j in range(self.count[b]):
            out[j] = (self.head[b] - self.count[b] + j) % self.N
        return out

    def context(self, b, layer, k_d, v_d):
        """Logical sequence of Proposition 1: [prefix ; ring in FIFO order ; dynamic]. Returns (K, V, n_prefix)."""
        if self.static_len[b] < 0:
            raise RuntimeError("static prefix never initialised")
        S = self.static_len[b]
        order = self.slot_map(b)[: self.count[b]]
        kc = np.concatenate([self.k_static[layer, b, :S], self.k_ring[layer, b, order], np.asarray(k_d, np.float32)])
        vc = np.concatenate([self.v_static[layer, b, :S], self.v_ring[layer, b, order], np.asarray(v_d, np.float32)])
        return kc, vc, S + self.count[b]

    def attention(self, b, layer, q, k_d, v_d, dyn_mask=0, scale=None, partitioned=False):
        """q [T][Hq][d], k_d/v_d [T][Hkv][d] -> [T][Hq][d] float64."""
        if partitioned:
            if self.static_len[b] < 0:
                raise RuntimeError("static prefix never initialised")
            return attention_part(q, self.k_static[layer, b], self.v_static[layer, b], self.static_len[b],
                                  self.k_ring[layer, b], self.v_ring[layer, b], self.head[b], self.count[b],
                                  k_d, v_d, dyn_mask, scale)
        kc, vc, n_prefix = self.context(b, layer, k_d, v_d)
        return attention_def(q, kc, vc, n_prefix, dyn_mask, scale)

    def attention_batched(self, layer, q, k_d, v_d, dyn_mask=0, scale=None, streams=None):
        """q [B][T][Hq][d] etc.; returns [len(streams)][T][Hq][d] float64."""
        streams = range(self.B) if streams is None else streams
        return np.stack([self.attention(b, layer, q[b], k_d[b], v_d[b], dyn_mask, scale) for b in streams])
