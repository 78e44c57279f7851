"""A whole action-expert denoising step built from the library's calls: per layer the adaptive norm folded into the
packed Q/K/V projection, the partitioned attention, the output projection with its residual, the adaptive norm folded
into the fused gate/up projections of the SwiGLU block and the down projection with its residual; then the velocity
head and the Euler update of the action chunk (Sec. 2.1, Sec. 3.1-3.3). The output and down projections with their
residual adds are reflex_linear_residual, and so are the two A-wide heads (input projection from the A = 32 action
dimensions, velocity head back to them; no residual): every contraction of the step runs in this package's kernels.

The paper does not print the expert's architecture; this is the usual pre-norm block of a pi0-class expert with both
norms adaptive, no biases and no positional term (positions are outside the path), written down so that the fused calls
can be timed inside the step they belong to.

    h = W_in a                                             (action chunk a [B][T][A] -> tokens [B][T][D])
    for l:  q, k, v = W_QKV,l AdaRMSNorm(h; gamma_{2l}(c));  o = PartitionedAttention_l(q, k, v);  h += W_O,l o
            m = SiLU(W_g,l n) * (W_u,l n), n = AdaRMSNorm(h; gamma_{2l+1}(c));                     h += W_D,l m
    v = W_out AdaRMSNorm(h; gamma_{2L}(c));   a <- a - v / K
"""
from __future__ import annotations

import torch

from . import binding as rb
from . import synth


class ActionExpert:
    def __init__(self, w: synth.Workload, cache: rb.Cache, weights: dict, F: int, device="cuda:0"):
        """weights: dict of torch tensors in the storage dtype (see expert_weights() for names and shapes)."""
        self.w, self.cache, self.F = w, cache, F
        self.dev = torch.device(device)
        self.tdt = rb.torch_dtype(w.dtype)
        self.W = weights
        B, T, D = w.B, w.T, w.D
        n_norm = 2 * w.L + 1
        self.n_norm = n_norm
        self.gates = torch.empty((n_norm * B * (D + w.Hd),), dtype=torch.float32, device=self.dev)
        e = lambda *s: torch.empty(s, dtype=self.tdt, device=self.dev)
        self.h, self.y = e(B, T, D), e(B, T, D)
        self.q, self.k, self.v = e(B, T, w.Hq, w.d), e(B, T, w.Hkv, w.d), e(B, T, w.Hkv, w.d)
        self.o = e(B, T, w.Hq, w.d)
        self.m = e(B, T, F)
        self.vel = e(B, T, w.A)
        self.a_lowp = e(B, T, w.A)

    def gate(self, i: int):
        w = self.w
        n = w.B * w.D
        return self.gates[i * n:(i + 1) * n].view(w.B, w.D)

    def step(self, a: torch.Tensor, cond: torch.Tensor, k: int, stream=None):
        """One Euler step on the fp32 action chunk a [B][T][A] (updated in place); cond [B][Cd] in the storage dtype."""
        w, W = self.w, self.W
        B, T, D = w.B, w.T, w.D
        rb.reflex_adarmsnorm_gate(cond, W["W1"], W["b1"], W["W2"], W["b2"], self.gates, stream=stream)   # all 2L + 1 gates
        self.a_lowp.copy_(a)
        rb.reflex_linear_residual(self.a_lowp.view(B * T, w.A), W["W_in"], None, self.h.view(B * T, D), cache=self.cache, stream=stream)
        for l in range(w.L):
            rb.reflex_adarmsnorm_qkv(self.h, self.gate(2 * l), W["Wqkv"][l], self.q, self.k, self.v, cache=self.cache, stream=stream)
            rb.reflex_partitioned_attention(self.cache, l, self.q, self.k, self.v, self.o, stream=stream)
            rb.reflex_linear_residual(self.o.view(B * T, w.Hq * w.d), W["Wo"][l], self.h, self.h, cache=self.cache, stream=stream)
            rb.reflex_adarmsnorm_swiglu(self.h, self.gate(2 * l + 1), W["Wgu"][l], self.m, cache=self.cache, stream=stream)
            rb.reflex_linear_residual(self.m.view(B * T, self.F), W["Wd"][l], self.h, self.h, cache=self.cache, stream=stream)
        rb.reflex_adarmsnorm(self.h, self.y, None, None, None, None, None, gate_buf=self.gate(2 * w.L), stream=stream)
        rb.reflex_linear_residual(self.y.view(B * T, D), W["W_out"], None, self.vel.view(B * T, w.A), cache=self.cache, stream=stream)
        rb.reflex_flow_step(a, self.vel, None, k, w.K, stream=stream)
        return a


def expert_weights(w: synth.Workload, F: int, std_scale: float = 1.0) -> dict:
    """Seeded weights as fp32 numpy arrays holding storage-representable values (the oracle and the device get the same bits).
    Projections are N(0, 1/fan_in), scaled by std_scale on the two residual branches' output projections."""
    L, D, A = w.L, w.D, w.A
    nq = w.Hq * w.d
    n_norm = 2 * L + 1
    g = lambda name, shape, std, layer=0: synth.normal(w, name, shape, layer, 7, std)
    out = {
        "W_in": g("misc", (D, A), A ** -0.5, 0), "W_out": g("misc", (A, D), D ** -0.5, 1),
        "Wqkv": g("Wqkv", (L, (w.Hq + 2 * w.Hkv) * w.d, D), D ** -0.5), "Wo": g("Wo", (L, D, nq), std_scale * nq ** -0.5),
        "Wgu": g("Wgu", (L, 2 * F, D), D ** -0.5), "Wd": g("misc", (L, D, F), std_scale * F ** -0.5, 2),
        "W1": g("W1", (n_norm, w.Hd, w.Cd), 0.02), "b1": g("b1", (n_norm, w.Hd), 0.1),
        "W2": g("W2", (n_norm, D, w.Hd), 0.02), "b2": g("b2", (n_norm, D), 0.1),
    }
    return out


def random_weights_device(w: synth.Workload, F: int, device="cuda:0", seed: int = 99) -> dict:
    """The same shapes as expert_weights(), drawn on the device (benchmarks: no host copy of 0.6 GB of weights)."""
    tdt = rb.torch_dtype(w.dtype)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    L, D, A = w.L, w.D, w.A
    nq, n_norm = w.Hq * w.d, 2 * w.L + 1
    r = lambda shape, std: (torch.randn(*shape, generator=g, device=device, dtype=torch.float32) * std).to(tdt).contiguous()
    return {"W_in": r((D, A), A ** -0.5), "W_out": r((A, D), D ** -0.5), "Wqkv": r((L, (w.Hq + 2 * w.Hkv) * w.d, D), D ** -0.5),
            "Wo": r((L, D, nq), 0.5 * nq ** -0.5), "Wgu": r((L, 2 * F, D), D ** -0.5), "Wd": r((L, D, F), 0.5 * F ** -0.5),
            "W1": r((n_norm, w.Hd, w.Cd), 0.02), "b1": r((n_norm, w.Hd), 0.1), "W2": r((n_norm, D, w.Hd), 0.02), "b2": r((n_norm, D), 0.1)}
