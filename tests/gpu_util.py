"""Helpers for the GPU parity tests: upload of storage-rounded arrays, tolerance checks, and a twin
driver that applies the same cache operation to the oracle and to the CUDA library."""
import numpy as np
import torch

from oracle import reflex_oracle as orc
from paper_2607_14695_b200 import binding as rb
from paper_2607_14695_b200 import synth

DEV = "cuda:0"

# bf16 storage: the contract's tolerances against the fp64 oracle
BF16_MAX_ABS = 2e-2
BF16_MEAN_ABS = 2e-3
# fp32 storage (tiny config): fp32 accumulation over <= a few hundred terms of O(1) magnitude
F32_MAX_ABS = 2e-5
F32_MEAN_ABS = 2e-6


def to_dev(a: np.ndarray, dtype: int) -> torch.Tensor:
    """fp32 array holding storage-representable values -> device tensor of the storage dtype (exact)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)
    return t.to(torch.bfloat16).contiguous() if dtype == synth.DTYPE_BF16 else t.contiguous()


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def check_close(got: np.ndarray, want: np.ndarray, dtype: int, what: str, rel_clause: bool = False, out_scale: float = 1.0):
    """max-abs / mean-abs contract. rel_clause adds the bf16 output-spacing allowance max(2e-2, 2^-7 |want|)
    used for normalised outliers (|y| >= 4 has a bf16 half-ulp above 2e-2 / 1.28). out_scale (>= 1) widens the mean-abs
    bound for outputs whose rms is that many times the unit variance the contract presumes (the spacing of the storage
    dtype grows with the magnitude); the element-wise bound is not widened."""
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    max_tol, mean_tol = (BF16_MAX_ABS, BF16_MEAN_ABS) if dtype == synth.DTYPE_BF16 else (F32_MAX_ABS, F32_MEAN_ABS)
    mean_tol *= max(1.0, float(out_scale))
    if rel_clause:
        lim = np.maximum(max_tol, 2.0 ** -7 * np.abs(want)) if dtype == synth.DTYPE_BF16 else np.maximum(max_tol, 1e-6 * np.abs(want))
        bad = err > lim
        assert not bad.any(), f"{what}: {bad.sum()} elements beyond max(tol, rel): worst {err.max():.3e}"
        base = err[np.abs(want) < 4.0]
        if base.size:
            assert base.mean() <= mean_tol, f"{what}: mean-abs {base.mean():.3e}"
    else:
        assert err.max() <= max_tol, f"{what}: max-abs {err.max():.3e} > {max_tol}"
        assert err.mean() <= mean_tol, f"{what}: mean-abs {err.mean():.3e} > {mean_tol}"
    return float(err.max()), float(err.mean())


class Twin:
    """The same partitioned cache on both sides: OracleCache (CPU) and rb.Cache (CUDA)."""

    def __init__(self, w: synth.Workload, head0=None, T_max=None, poison=False, static_banks=1):
        self.w = w
        self.o = orc.OracleCache(w.L, w.B, w.Hkv, w.d, w.S_max, w.N, head0=head0)
        self.g = rb.Cache(w.L, w.B, w.Hq, w.Hkv, w.d, w.S_max, w.N, T_max or w.T, w.dtype, device=DEV,
                          ring_head0=None if head0 is None else [int(h) for h in head0], static_banks=static_banks)
        self.bank = [0] * w.B       # which static bank of the slab holds each stream's current prefix
        if poison:  # stale / empty rows hold NaN on both sides: any read of them shows up
            self.g.k_slab.fill_(float("nan")); self.g.v_slab.fill_(float("nan"))
            for a in (self.o.k_static, self.o.v_static, self.o.k_ring, self.o.v_ring):
                a[:] = np.nan

    def init_static(self, ids, S_list, variant=0, S_src=None):
        w = self.w
        S_src = max(S_list) if S_src is None else S_src
        ks = synth.normal(w, "k_static", (len(ids), w.L, S_src, w.Hkv, w.d), 0, variant)
        vs = synth.normal(w, "v_static", (len(ids), w.L, S_src, w.Hkv, w.d), 0, variant)
        for i, b in enumerate(ids):
            self.o.init_static(b, ks[i][:, : S_list[i]], vs[i][:, : S_list[i]])
        rb.reflex_cache_init_static(self.g, ids, to_dev(ks, w.dtype), to_dev(vs, w.dtype), S=S_list)

    def stage_static(self, ids, S_list, variant, stream=None):
        """A new prefix for these streams goes to the bank that is not being read, on both sides."""
        w = self.w
        S_src = max(S_list)
        ks = synth.normal(w, "k_static", (len(ids), w.L, S_src, w.Hkv, w.d), 0, variant)
        vs = synth.normal(w, "v_static", (len(ids), w.L, S_src, w.Hkv, w.d), 0, variant)
        for i, b in enumerate(ids):
            self.o.stage_static(b, ks[i][:, : S_list[i]], vs[i][:, : S_list[i]])
        dk, dv = to_dev(ks, w.dtype), to_dev(vs, w.dtype)
        rb.reflex_cache_stage_static(self.g, ids, dk, dv, S=S_list, stream=stream)
        return dk, dv        # (kept alive by the caller while a side stream may still read them)

    def commit_static(self, ids, stream=None):
        for b in ids:
            self.o.commit_static(b)
            self.bank[b] ^= 1
        rb.reflex_cache_commit_static(self.g, ids, stream=stream)

    def append(self, ids, m, variant):
        w = self.w
        kn = synth.normal(w, "k_new", (len(ids), w.L, m, w.Hkv, w.d), 0, variant)
        vn = synth.normal(w, "v_new", (len(ids), w.L, m, w.Hkv, w.d), 0, variant)
        ev_o = [self.o.append_sliding(b, kn[i], vn[i]) for i, b in enumerate(ids)]
        ev_g = rb.reflex_cache_append_sliding(self.g, ids, to_dev(kn, w.dtype), to_dev(vn, w.dtype))
        assert ev_g == ev_o, (ev_g, ev_o)
        return ev_o

    def check_state(self):
        """Ring indices, slot maps and cache bytes are compared exactly."""
        w = self.w
        sl, hd, ct, tot = rb.reflex_cache_get_state(self.g)
        assert sl == list(self.o.static_len) and hd == list(self.o.head) and ct == list(self.o.count) and tot == list(self.o.total)
        ks = self.g.k_slab.float().cpu().numpy(); vs = self.g.v_slab.float().cpu().numpy()
        for b in range(w.B):
            assert rb.reflex_cache_slot_map(self.g, b) == self.o.slot_map(b)
            S = max(self.o.static_len[b], 0)
            s0 = self.bank[b] * w.S_max
            assert np.array_equal(ks[:, b, s0:s0 + S], self.o.k_static[:, b, :S]) and np.array_equal(vs[:, b, s0:s0 + S], self.o.v_static[:, b, :S])
            live = self.o.slot_map(b)[: self.o.count[b]]
            r0 = self.g.ring_off
            assert np.array_equal(ks[:, b, r0:][:, live], self.o.k_ring[:, b, live])
            assert np.array_equal(vs[:, b, r0:][:, live], self.o.v_ring[:, b, live])

    def attention(self, layer, variant, dyn_mask=0, T=None, streams=None, scale=0.0, what="attention", partitioned=False, q_scale=1.0, rel_clause=False):
        w = self.w
        T = w.T if T is None else T
        q = synth.normal(w, "q", (w.B, T, w.Hq, w.d), layer, variant)
        if q_scale != 1.0:   # wider logits (the same rounding to the storage dtype on both sides)
            q = synth.round_storage(q * np.float32(q_scale), w.dtype)
        kd = synth.normal(w, "k_dyn", (w.B, T, w.Hkv, w.d), layer, variant)
        vd = synth.normal(w, "v_dyn", (w.B, T, w.Hkv, w.d), layer, variant)
        out = torch.full((w.B, T, w.Hq, w.d), float("nan"), dtype=rb.torch_dtype(w.dtype), device=DEV)
        rb.reflex_partitioned_attention(self.g, layer, to_dev(q, w.dtype), to_dev(kd, w.dtype), to_dev(vd, w.dtype), out,
                                        scale=scale, dyn_mask=dyn_mask)
        rb.reflex_cache_check_status(self.g)   # no bounded device-side wait ran out
        got = to_host(out)
        if not np.isfinite(got).all():
            bad = np.argwhere(~np.isfinite(got))
            raise AssertionError(f"{what}: non-finite output, {len(bad)} elements; streams {np.unique(bad[:, 0])[:8]}, tokens {np.unique(bad[:, 1])[:12]}, "
                                 f"heads {np.unique(bad[:, 2])}, columns {np.unique(bad[:, 3])[:6]}..{bad[:, 3].max()} ({len(np.unique(bad[:, 3]))})")
        streams = list(range(w.B)) if streams is None else streams
        res = []
        for b in streams:
            want = self.o.attention(b, layer, q[b], kd[b], vd[b], dyn_mask, None if scale <= 0 else scale, partitioned=partitioned)
            res.append(check_close(got[b], want, w.dtype, f"{what} stream {b} layer {layer}", rel_clause=rel_clause))
        return res
