"""Seeded synthetic inputs for the Reflex hot path (shared by the tests, the bench and the smoke check).

This module holds workload shapes and random-input recipes only. It contains none of the
method's arithmetic (no normalisation, attention, ring or flow-update code): both the CUDA
path and the CPU oracle receive the arrays it produces, bit for bit.

Value recipe (stands in for the paper's LIBERO/Kinetix + Pi0-class workloads, which need
simulators and trained weights): activations are standard normal, because the paper's own
stress case is the flow state x ~ N(0, I) at t = 1 (Sec. 3.2); shapes follow a pi0-class
action expert (chunk of 50 action tokens, 10 flow steps, Appendix C).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

DTYPE_BF16 = 0
DTYPE_F32 = 1


@dataclass(frozen=True)
class Workload:
    """Shapes of one configuration. Symbols: B streams, L layers, Hq/Hkv query/KV heads,
    d head_dim, S static-prefix tokens (S_max capacity), N ring slots, T dynamic action tokens,
    D AdaRMSNorm width, Cd conditioning width, Hd gate-MLP hidden width, A action width,
    K denoising (Euler) steps, m tokens appended per control tick."""
    name: str
    seed: int
    dtype: int
    B: int
    L: int
    Hq: int
    Hkv: int
    d: int
    S: int
    S_max: int
    N: int
    T: int
    D: int
    Cd: int
    Hd: int
    A: int
    K: int
    m: int = 1
    ticks: int = 1
    outlier_frac: float = 0.0
    outlier_mult: float = 1.0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS = {
    # tiny fp32 single-layer check, 40 ticks of 4 Euler steps
    "cfg1": Workload("cfg1", 0, DTYPE_F32, B=1, L=1, Hq=2, Hkv=1, d=64, S=64, S_max=64, N=16, T=8,
                     D=128, Cd=40, Hd=32, A=8, K=4, ticks=40),
    # one pi0-class layer, batch 1
    "cfg2": Workload("cfg2", 1, DTYPE_BF16, B=1, L=1, Hq=8, Hkv=1, d=256, S=816, S_max=816, N=32, T=50,
                     D=1024, Cd=288, Hd=256, A=32, K=10),
    # 18-layer action-expert stack streamed at 50 Hz, batch 1
    "cfg3": Workload("cfg3", 2, DTYPE_BF16, B=1, L=18, Hq=8, Hkv=1, d=256, S=816, S_max=816, N=32, T=50,
                     D=1024, Cd=288, Hd=256, A=32, K=10, ticks=500),
    # batched serving, 64 independent streams (the HBM-roofline configuration)
    "cfg4": Workload("cfg4", 3, DTYPE_BF16, B=64, L=18, Hq=8, Hkv=1, d=256, S=816, S_max=816, N=32, T=50,
                     D=1024, Cd=288, Hd=256, A=32, K=10),
    # long-context stress with outliers in the norm input
    "cfg5": Workload("cfg5", 4, DTYPE_BF16, B=16, L=18, Hq=8, Hkv=1, d=256, S=4160, S_max=4160, N=256, T=50,
                     D=1024, Cd=288, Hd=256, A=32, K=10, outlier_frac=1e-3, outlier_mult=1e3),
}

# tensor ids for the seed sequence
TID = {"k_static": 1, "v_static": 2, "k_new": 3, "v_new": 4, "q": 5, "k_dyn": 6, "v_dyn": 7, "x": 8,
       "cond_state": 9, "W1": 10, "b1": 11, "W2": 12, "b2": 13, "v_flow": 14, "noise": 15, "head0": 16,
       "outlier_mask": 17, "misc": 18, "Wqkv": 19, "Wo": 20, "Wgu": 21}


def rng_for(w_or_seed, tensor: str, layer: int = 0, variant: int = 0) -> np.random.Generator:
    seed = w_or_seed.seed if isinstance(w_or_seed, Workload) else int(w_or_seed)
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, TID[tensor], layer, variant])))


# ---- storage-dtype rounding (input preparation, shared bit for bit by both sides) ----

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16). NaN/Inf pass through."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    naninf = (u & 0x7F800000) == 0x7F800000
    out = np.where(naninf, u >> 16, rounded).astype(np.uint16)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def round_storage(a: np.ndarray, dtype: int) -> np.ndarray:
    """Round an fp32 array once to the storage dtype; result is fp32 holding exactly representable values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == DTYPE_F32:
        return a
    return bf16_bits_to_f32(f32_to_bf16_bits(a))


def normal(w: Workload, tensor: str, shape, layer: int = 0, variant: int = 0, std: float = 1.0) -> np.ndarray:
    """Seeded N(0, std^2) tensor rounded to the workload's storage dtype (returned as fp32)."""
    g = rng_for(w, tensor, layer, variant)
    a = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a = a * np.float32(std)
    return round_storage(a, w.dtype)


def norm_input(w: Workload, layer: int, variant: int, B: int | None = None) -> np.ndarray:
    """x for AdaRMSNorm, [B][T][D]; N(0,1) plus (cfg5) a seeded Bernoulli mask of x1e3 outliers."""
    B = w.B if B is None else B
    g = rng_for(w, "x", layer, variant)
    a = g.standard_normal(size=(B, w.T, w.D), dtype=np.float32)
    if w.outlier_frac > 0.0:
        gm = rng_for(w, "outlier_mask", layer, variant)
        mask = gm.random(size=a.shape) < w.outlier_frac
        a = np.where(mask, a * np.float32(w.outlier_mult), a).astype(np.float32)
    return round_storage(a, w.dtype)


# ---- conditioning vector c = [emb(t_k), s_t], built by the caller of the library ----

def timestep_embedding(t: float, dim: int) -> np.ndarray:
    """Sinusoidal embedding of the flow time t in [0,1]: sin/cos over geometrically spaced periods.
    The paper does not fix the formula; parity does not depend on it because both sides get the same bits."""
    half = dim // 2
    periods = 4e-3 * (4.0 / 4e-3) ** (np.arange(half, dtype=np.float64) / max(half - 1, 1))
    ang = 2.0 * np.pi * float(t) / periods
    return np.concatenate([np.sin(ang), np.cos(ang)]).astype(np.float32)


def cond_vectors(w: Workload, t: float, B: int | None = None, variant: int = 0) -> np.ndarray:
    """[B][Cd] conditioning: timestep embedding of t followed by a seeded proprio state per stream."""
    B = w.B if B is None else B
    state_dim = 8 if w.Cd <= 64 else 32
    emb = timestep_embedding(t, w.Cd - state_dim)
    g = rng_for(w, "cond_state", 0, variant)
    s = g.standard_normal(size=(B, state_dim), dtype=np.float32)
    c = np.concatenate([np.broadcast_to(emb, (B, emb.shape[0])), s], axis=1)
    return round_storage(c, w.dtype)


def gate_weights(w: Workload, layer: int, std: float = 0.02, bias_std: float = 0.1):
    """Gate-MLP parameters W1[Hd][Cd], b1[Hd], W2[D][Hd], b2[D] of Eq. 2: N(0, std^2) weights and N(0, bias_std^2)
    biases, all rounded to the storage dtype. With the defaults the gate 1 + MLP(c) stays within about 1 +- 0.3 and
    both biases move it visibly; a larger std makes the hidden layer and the second product carry the gate."""
    W1 = normal(w, "W1", (w.Hd, w.Cd), layer, 0, std)
    W2 = normal(w, "W2", (w.D, w.Hd), layer, 0, std)
    if bias_std > 0.0:
        b1 = normal(w, "b1", (w.Hd,), layer, 0, bias_std)
        b2 = normal(w, "b2", (w.D,), layer, 0, bias_std)
    else:
        b1 = np.zeros((w.Hd,), np.float32)
        b2 = np.zeros((w.D,), np.float32)
    return W1, b1, W2, b2


def qkv_weights(w: Workload, layer: int) -> np.ndarray:
    """Packed projection W_QKV = [W_Q; W_K; W_V], [(Hq + 2 Hkv) d][D], N(0, 1/D): unit-variance outputs for unit-variance inputs."""
    return normal(w, "Wqkv", ((w.Hq + 2 * w.Hkv) * w.d, w.D), layer, 0, float(w.D) ** -0.5)


def swiglu_weights(w: Workload, layer: int, F: int) -> np.ndarray:
    """[W_gate; W_up] of a SwiGLU block, [2F][D], N(0, 1/D)."""
    return normal(w, "Wgu", (2 * F, w.D), layer, 0, float(w.D) ** -0.5)


def ring_head0(w: Workload, B: int | None = None) -> np.ndarray:
    """Per-stream random initial ring write positions in [0, N)."""
    B = w.B if B is None else B
    return rng_for(w, "head0").integers(0, w.N, size=(B,), dtype=np.int32)
