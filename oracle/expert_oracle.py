"""Oracle of the whole action-expert denoising step. TEST INFRASTRUCTURE ONLY.

The step chained in double precision from the oracle's own pieces (adaptive norm + packed projection, attention by
definition, adaptive norm + SwiGLU projections, Euler update) and plain numpy matrix products for the four plain
projections; nothing is rounded in between (the residual stream, Q/K/V and all intermediates stay in double and are
handed to the C routines as float32 only where those take float32)."""
import numpy as np

from . import reflex_oracle as orc


def expert_step(ocache: "orc.OracleCache", W: dict, a: np.ndarray, cond: np.ndarray, K: int, Hq: int, Hkv: int, d: int, F: int,
                eps: float = 1e-6, dyn_mask: int = 0, streams=None):
    """a [B][T][A] float64 (returned updated), cond [B][Cd]. Returns (a_new, v). streams: compute these streams only (the
    streams are independent; the others keep their chunk and a zero velocity)."""
    B, T, A = a.shape
    L = W["Wqkv"].shape[0]
    f64 = lambda x: np.asarray(x, np.float64)
    f32 = lambda x: np.asarray(x, np.float32)
    a_new = a.copy()
    v_all = np.zeros_like(a)
    for b in (range(B) if streams is None else streams):
        h = a[b] @ f64(W["W_in"]).T                                             # [T][D]
        for l in range(L):
            g1 = (W["W1"][2 * l], W["b1"][2 * l], W["W2"][2 * l], W["b2"][2 * l])
            q, k, v = orc.adarmsnorm_qkv(f32(h), cond[b], *g1, W["Wqkv"][l], Hq, Hkv, d, eps)
            o = ocache.attention(b, l, f32(q), f32(k), f32(v), dyn_mask, None)
            h = h + o.reshape(T, Hq * d) @ f64(W["Wo"][l]).T
            g2 = (W["W1"][2 * l + 1], W["b1"][2 * l + 1], W["W2"][2 * l + 1], W["b2"][2 * l + 1])
            m = orc.adarmsnorm_swiglu(f32(h), cond[b], *g2, W["Wgu"][l][:F], W["Wgu"][l][F:], eps)
            h = h + m @ f64(W["Wd"][l]).T
        gf = (W["W1"][2 * L], W["b1"][2 * L], W["W2"][2 * L], W["b2"][2 * L])
        y = orc.adarmsnorm(f32(h), cond[b], *gf, eps)
        v_all[b] = y @ f64(W["W_out"]).T
    x = np.ascontiguousarray(a_new, np.float64)
    orc.flow_step(x, v_all.astype(np.float32), K)      # (the velocity handed over as float32, as the routine takes it)
    return x, v_all
