"""Thin ctypes binding over libreflex_b200.so, same names as the C ABI in include/reflex.h.

Argument marshalling only: every step of the hot path runs in the library's CUDA kernels. torch is
used for device memory and streams. There is no CPU fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libreflex_b200.so")

DTYPE_BF16 = 0
DTYPE_F32 = 1
ATTN_AUTO, ATTN_SIMT, ATTN_TC, ATTN_TC2 = 0, 1, 2, 3

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGN, ERR_STATE, ERR_CUDA, ERR_TIMEOUT, ERR_NOT_IMPLEMENTED = -1, -2, -3, -4, -5, -6, -7

EXPORTS = [
    "reflex_last_error_string", "reflex_version", "reflex_kernel_launch_count", "reflex_cache_slab_bytes", "reflex_workspace_bytes",
    "reflex_cache_create", "reflex_cache_destroy", "reflex_cache_get_state", "reflex_cache_slot_map",
    "reflex_cache_set_attention_impl", "reflex_cache_check_status", "reflex_cache_selftest_wait_limit", "reflex_cache_init_static", "reflex_cache_stage_static",
    "reflex_cache_commit_static", "reflex_cache_append_sliding",
    "reflex_adarmsnorm", "reflex_adarmsnorm_gate", "reflex_adarmsnorm_noalloc", "reflex_adarmsnorm_qkv", "reflex_adarmsnorm_swiglu", "reflex_linear_residual", "reflex_partitioned_attention",
    "reflex_flow_step", "reflex_overlap_create", "reflex_overlap_destroy", "reflex_overlap_tick", "reflex_overlap_inference_done",
    "reflex_overlap_simulate",
]


class OverlapEvent(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("chunk", "action", "launch_now", "stalled", "lookahead", "reserved")] + [("stalls_total", ctypes.c_int64)]


class OverlapStats(ctypes.Structure):
    _fields_ = [("chunks", ctypes.c_int64), ("stall_ticks", ctypes.c_int64), ("stall_time_s", ctypes.c_double), ("total_time_s", ctypes.c_double),
                ("mean_staleness_s", ctypes.c_double), ("mean_lookahead", ctypes.c_double), ("min_lookahead", ctypes.c_int32),
                ("max_lookahead", ctypes.c_int32)]


class CacheDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("L", "B", "Hq", "Hkv", "d", "S_max", "N", "T_max", "dtype", "static_banks")]


class ReflexError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"reflex error {code}: {msg}")
        self.code = code


_lib = None


def load():
    """Load the C-ABI library (raises if it has not been built: there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_14695_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    i32p, i64p = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)
    dp = ctypes.POINTER(CacheDesc)
    lib.reflex_last_error_string.restype = ctypes.c_char_p
    lib.reflex_version.restype = ctypes.c_char_p
    lib.reflex_kernel_launch_count.restype = ctypes.c_ulonglong
    lib.reflex_cache_slab_bytes.argtypes = [dp]; lib.reflex_cache_slab_bytes.restype = ctypes.c_size_t
    lib.reflex_workspace_bytes.argtypes = [dp]; lib.reflex_workspace_bytes.restype = ctypes.c_size_t
    lib.reflex_cache_create.argtypes = [dp, vp, vp, vp, i32p, vp, ctypes.POINTER(vp)]
    lib.reflex_cache_destroy.argtypes = [vp]
    lib.reflex_cache_get_state.argtypes = [vp, i32p, i32p, i32p, i64p, vp]
    lib.reflex_cache_slot_map.argtypes = [vp, i, i32p]
    lib.reflex_cache_set_attention_impl.argtypes = [vp, i]
    lib.reflex_cache_check_status.argtypes = [vp, vp]
    lib.reflex_cache_selftest_wait_limit.argtypes = [vp, i, vp]
    lib.reflex_cache_init_static.argtypes = [vp, i32p, i, vp, vp, i, i32p, vp]
    lib.reflex_cache_stage_static.argtypes = [vp, i32p, i, vp, vp, i, i32p, vp]
    lib.reflex_cache_commit_static.argtypes = [vp, i32p, i, vp]
    lib.reflex_cache_append_sliding.argtypes = [vp, i32p, i, vp, vp, i, i32p, vp]
    lib.reflex_adarmsnorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp]
    lib.reflex_adarmsnorm_gate.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, vp]
    lib.reflex_adarmsnorm_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp]
    lib.reflex_adarmsnorm_qkv.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, i, vp]
    lib.reflex_adarmsnorm_swiglu.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, f, i, i, vp]
    lib.reflex_linear_residual.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, vp]
    lib.reflex_partitioned_attention.argtypes = [vp, i, vp, vp, vp, vp, i, f, i, vp]
    lib.reflex_flow_step.argtypes = [vp, vp, vp, i, i, i, i, i, i, vp]
    dbl = ctypes.c_double
    lib.reflex_overlap_create.argtypes = [i, dbl, dbl, ctypes.POINTER(vp)]
    lib.reflex_overlap_destroy.argtypes = [vp]
    lib.reflex_overlap_tick.argtypes = [vp, ctypes.POINTER(OverlapEvent)]
    lib.reflex_overlap_inference_done.argtypes = [vp, dbl]
    lib.reflex_overlap_simulate.argtypes = [i, dbl, dbl, ctypes.POINTER(dbl), i, i, i, ctypes.POINTER(OverlapStats)]
    for name in EXPORTS:
        getattr(lib, name)  # every declared symbol must resolve
    _lib = lib
    return lib


def _check(rc: int):
    if rc != OK:
        raise ReflexError(rc, load().reflex_last_error_string().decode())


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _i32(seq: Optional[Sequence[int]]):
    if seq is None:
        return None
    return (ctypes.c_int32 * len(seq))(*[int(v) for v in seq])


def torch_dtype(dtype: int) -> torch.dtype:
    return torch.bfloat16 if dtype == DTYPE_BF16 else torch.float32


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float32:
        return DTYPE_F32
    raise ValueError(f"unsupported storage dtype {t.dtype}")


def reflex_version() -> str:
    return load().reflex_version().decode()


def reflex_kernel_launch_count() -> int:
    return int(load().reflex_kernel_launch_count())


def reflex_cache_slab_bytes(desc: CacheDesc) -> int:
    return int(load().reflex_cache_slab_bytes(ctypes.byref(desc)))


def reflex_workspace_bytes(desc: CacheDesc) -> int:
    return int(load().reflex_workspace_bytes(ctypes.byref(desc)))


class Cache:
    """Owns the device memory the library borrows (two slabs + workspace, allocated once through
    torch) and the opaque handle."""

    def __init__(self, L, B, Hq, Hkv, d, S_max, N, T_max, dtype, device="cuda:0", ring_head0=None, stream=None, static_banks=1):
        lib = load()
        self.desc = CacheDesc(L, B, Hq, Hkv, d, S_max, N, T_max, dtype, static_banks)
        self.ring_off = (2 if static_banks == 2 else 1) * S_max     # first ring row of a (layer, stream) block
        slab = reflex_cache_slab_bytes(self.desc)
        wsb = reflex_workspace_bytes(self.desc)
        if slab == 0 or wsb == 0:
            raise ReflexError(ERR_SHAPE, "invalid cache descriptor")
        self.device = torch.device(device)
        tdt = torch_dtype(dtype)
        self.k_slab = torch.zeros((L, B, self.ring_off + N, Hkv, d), dtype=tdt, device=self.device)
        self.v_slab = torch.zeros_like(self.k_slab)
        assert self.k_slab.numel() * self.k_slab.element_size() == slab
        self.workspace = torch.zeros((wsb,), dtype=torch.uint8, device=self.device)
        self.handle = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib.reflex_cache_create(ctypes.byref(self.desc), _ptr(self.k_slab), _ptr(self.v_slab), _ptr(self.workspace),
                                           _i32(ring_head0), _stream(stream), ctypes.byref(self.handle)))

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle:
            load().reflex_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def reflex_cache_get_state(cache: Cache, stream=None):
    B = cache.desc.B
    sl, hd, ct = (ctypes.c_int32 * B)(), (ctypes.c_int32 * B)(), (ctypes.c_int32 * B)()
    tot = (ctypes.c_int64 * B)()
    _check(load().reflex_cache_get_state(cache.handle, sl, hd, ct, tot, _stream(stream)))
    return list(sl), list(hd), list(ct), list(tot)


def reflex_cache_slot_map(cache: Cache, b: int):
    out = (ctypes.c_int32 * cache.desc.N)()
    _check(load().reflex_cache_slot_map(cache.handle, int(b), out))
    return list(out)


def reflex_cache_set_attention_impl(cache: Cache, impl: int):
    _check(load().reflex_cache_set_attention_impl(cache.handle, int(impl)))


def reflex_cache_check_status(cache: Cache, stream=None):
    _check(load().reflex_cache_check_status(cache.handle, _stream(stream)))


def reflex_cache_selftest_wait_limit(cache: Cache, limit_us: int = 2000, stream=None):
    """Launch the bounded-wait probe: its wait runs out after limit_us and raises the cache's status word."""
    _check(load().reflex_cache_selftest_wait_limit(cache.handle, int(limit_us), _stream(stream)))


def reflex_cache_init_static(cache: Cache, stream_ids, k_static, v_static, S=None, stream=None):
    """k_static, v_static: device [n][L][S_src][Hkv][d]."""
    n = len(stream_ids)
    S_src = int(k_static.shape[2]) if k_static is not None else 0
    _check(load().reflex_cache_init_static(cache.handle, _i32(stream_ids), n, _ptr(k_static), _ptr(v_static), S_src,
                                           _i32(S), _stream(stream)))


def reflex_cache_stage_static(cache: Cache, stream_ids, k_static, v_static, S=None, stream=None):
    """Write a new prefix into the static bank that attention is not reading (cache created with static_banks=2)."""
    n = len(stream_ids)
    S_src = int(k_static.shape[2]) if k_static is not None else 0
    _check(load().reflex_cache_stage_static(cache.handle, _i32(stream_ids), n, _ptr(k_static), _ptr(v_static), S_src,
                                            _i32(S), _stream(stream)))


def reflex_cache_commit_static(cache: Cache, stream_ids, stream=None):
    """Make the staged prefix of these streams the one attention reads (index flip on `stream`)."""
    _check(load().reflex_cache_commit_static(cache.handle, _i32(stream_ids), len(stream_ids), _stream(stream)))


def reflex_cache_append_sliding(cache: Cache, stream_ids, k_new, v_new, stream=None):
    """k_new, v_new: device [n][L][m][Hkv][d]. Returns the per-stream eviction counts."""
    n = len(stream_ids)
    m = int(k_new.shape[2])
    ev = (ctypes.c_int32 * n)()
    _check(load().reflex_cache_append_sliding(cache.handle, _i32(stream_ids), n, _ptr(k_new), _ptr(v_new), m, ev, _stream(stream)))
    return list(ev)


def reflex_adarmsnorm(x, y, cond, W1, b1, W2, b2, gate_buf=None, eps=1e-6, stream=None):
    """x, y [B][R][D]; cond [B][Cd] or None (then gate_buf [B][D] fp32 is the precomputed gate).
    With cond given, gate_buf (optional) must hold B*(D+Hd) floats: gate, then hidden-layer scratch."""
    B, R, D = x.shape
    Hd, Cd = (W1.shape if W1 is not None else (0, 0))
    _check(load().reflex_adarmsnorm(_ptr(x), _ptr(y), _ptr(cond), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(gate_buf),
                                    B, R, D, int(Cd), int(Hd), float(eps), dtype_code(x), _stream(stream)))
    return y


def _gate_dims(cond, W1, W2):
    """(L, B, D, Cd, Hd) from cond [B][Cd] and W1 [Hd][Cd] or stacked [L][Hd][Cd], W2 [D][Hd] or [L][D][Hd]."""
    B, Cd = cond.shape
    L = W1.shape[0] if W1.dim() == 3 else 1
    return L, B, int(W2.shape[-2]), int(Cd), int(W1.shape[-2])


def reflex_adarmsnorm_gate(cond, W1, b1, W2, b2, gate_buf, stream=None):
    """gate_buf[:L*B*D] <- 1 + W2_l SiLU(W1_l c + b1_l) + b2_l (fp32) for the L stacked layers; gate_buf holds
    L*B*(D+Hd) floats."""
    L, B, D, Cd, Hd = _gate_dims(cond, W1, W2)
    _check(load().reflex_adarmsnorm_gate(_ptr(cond), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(gate_buf), L, B, D, Cd, Hd,
                                         dtype_code(cond), _stream(stream)))
    return gate_buf


def reflex_adarmsnorm_noalloc(x, y, cond, W1, b1, W2, b2, eps=1e-6, stream=None):
    """AdaRMSNorm for callers that have no scratch buffer to lend: the gate scratch is an array inside the library
    (B*(D+Hd) <= 98304 floats). Calls on one device share that array, so calls that overlap on the GPU race."""
    B, R, D = x.shape
    Hd, Cd = W1.shape
    _check(load().reflex_adarmsnorm_noalloc(_ptr(x), _ptr(y), _ptr(cond), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2),
                                            B, R, D, int(Cd), int(Hd), float(eps), dtype_code(x), _stream(stream)))
    return y


def reflex_adarmsnorm_qkv(x, gate, Wqkv, q, k_dyn, v_dyn, eps=1e-6, impl=0, cache=None, stream=None):
    """x [B][R][D], gate fp32 [B][D], Wqkv [(Hq + 2 Hkv) d][D] -> q [B][R][Hq][d], k_dyn / v_dyn [B][R][Hkv][d]."""
    B, R, D = x.shape
    Hq, d = int(q.shape[2]), int(q.shape[3])
    Hkv = int(k_dyn.shape[2])
    _check(load().reflex_adarmsnorm_qkv(cache.handle if cache is not None else None, _ptr(x), _ptr(gate), _ptr(Wqkv), _ptr(q), _ptr(k_dyn),
                                        _ptr(v_dyn), B, R, D, Hq, Hkv, d, float(eps), dtype_code(x), int(impl), _stream(stream)))
    return q, k_dyn, v_dyn


def reflex_partitioned_attention(cache: Cache, layer, q, k_dyn, v_dyn, out, scale=0.0, dyn_mask=0, stream=None):
    """q, out [B][T][Hq][d]; k_dyn, v_dyn [B][T][Hkv][d]."""
    T = int(q.shape[1])
    _check(load().reflex_partitioned_attention(cache.handle, int(layer), _ptr(q), _ptr(k_dyn), _ptr(v_dyn), _ptr(out), T,
                                               float(scale), int(dyn_mask), _stream(stream)))
    return out


def reflex_flow_step(x, v, x_lowp, k, K, stream=None):
    """x [B][T][A] fp32 in place; v [B][T][A] storage dtype; x_lowp optional mirror."""
    B, T, A = x.shape
    _check(load().reflex_flow_step(_ptr(x), _ptr(v), _ptr(x_lowp), B, T, A, int(k), int(K), dtype_code(v), _stream(stream)))
    return x


# ---- prepared calls: arguments marshalled once, then replayed with ~1 us of host overhead per call ----

def stream_handle(stream=None) -> ctypes.c_void_p:
    """ctypes handle of a torch stream (default: the current one), for the prepared calls below."""
    return _stream(stream)


def _prepared(fn, args):
    lib = load()

    def call(stream: ctypes.c_void_p):
        rc = fn(*args, stream)
        if rc != OK:
            raise ReflexError(rc, lib.reflex_last_error_string().decode())

    return call


def prepare_adarmsnorm(x, y, cond, W1, b1, W2, b2, gate_buf=None, eps=1e-6):
    B, R, D = x.shape
    Hd, Cd = (W1.shape if W1 is not None else (0, 0))
    args = (_ptr(x), _ptr(y), _ptr(cond), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(gate_buf), B, R, D, int(Cd), int(Hd),
            float(eps), dtype_code(x))
    return _prepared(load().reflex_adarmsnorm, args)


def prepare_adarmsnorm_gate(cond, W1, b1, W2, b2, gate_buf):
    L, B, D, Cd, Hd = _gate_dims(cond, W1, W2)
    args = (_ptr(cond), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(gate_buf), L, B, D, Cd, Hd, dtype_code(cond))
    return _prepared(load().reflex_adarmsnorm_gate, args)


def reflex_adarmsnorm_swiglu(x, gate, Wgu, h, eps=1e-6, impl=0, cache=None, stream=None):
    """x [B][R][D], gate fp32 [B][D], Wgu [2F][D] = [W_gate; W_up] -> h [B][R][F] = SiLU(y W_gate^T) * (y W_up^T)."""
    B, R, D = x.shape
    F = int(h.shape[2])
    _check(load().reflex_adarmsnorm_swiglu(cache.handle if cache is not None else None, _ptr(x), _ptr(gate), _ptr(Wgu), _ptr(h), B, R, D, F,
                                           float(eps), dtype_code(x), int(impl), _stream(stream)))
    return h


def reflex_linear_residual(a, W, res, out, impl=0, cache=None, stream=None):
    """a [..., K] (all leading axes are rows), W [N][K], res [..., N] or None -> out [..., N] = res + a W^T; out may be res."""
    K, N = int(a.shape[-1]), int(W.shape[0])
    M = a.numel() // K
    _check(load().reflex_linear_residual(cache.handle if cache is not None else None, _ptr(a), _ptr(W), _ptr(res), _ptr(out), M, K, N,
                                         dtype_code(a), int(impl), _stream(stream)))
    return out


def prepare_linear_residual(a, W, res, out, impl=0, cache=None):
    K, N = int(a.shape[-1]), int(W.shape[0])
    args = (cache.handle if cache is not None else None, _ptr(a), _ptr(W), _ptr(res), _ptr(out), a.numel() // K, K, N, dtype_code(a), int(impl))
    return _prepared(load().reflex_linear_residual, args)


def prepare_adarmsnorm_swiglu(x, gate, Wgu, h, eps=1e-6, impl=0, cache=None):
    B, R, D = x.shape
    args = (cache.handle if cache is not None else None, _ptr(x), _ptr(gate), _ptr(Wgu), _ptr(h), B, R, D, int(h.shape[2]), float(eps),
            dtype_code(x), int(impl))
    return _prepared(load().reflex_adarmsnorm_swiglu, args)


def prepare_adarmsnorm_qkv(x, gate, Wqkv, q, k_dyn, v_dyn, eps=1e-6, impl=0, cache=None):
    B, R, D = x.shape
    args = (cache.handle if cache is not None else None, _ptr(x), _ptr(gate), _ptr(Wqkv), _ptr(q), _ptr(k_dyn), _ptr(v_dyn), B, R, D,
            int(q.shape[2]), int(k_dyn.shape[2]), int(q.shape[3]), float(eps), dtype_code(x), int(impl))
    return _prepared(load().reflex_adarmsnorm_qkv, args)


def prepare_partitioned_attention(cache: Cache, layer, q, k_dyn, v_dyn, out, scale=0.0, dyn_mask=0):
    args = (cache.handle, int(layer), _ptr(q), _ptr(k_dyn), _ptr(v_dyn), _ptr(out), int(q.shape[1]), float(scale), int(dyn_mask))
    return _prepared(load().reflex_partitioned_attention, args)


def prepare_flow_step(x, v, x_lowp, k, K):
    B, T, A = x.shape
    args = (_ptr(x), _ptr(v), _ptr(x_lowp), B, T, A, int(k), int(K), dtype_code(v))
    return _prepared(load().reflex_flow_step, args)


# ---- Algorithm 1: overlap scheduling (host logic) ----
class OverlapScheduler:
    """Thin wrapper over reflex_overlap_*: tick() once per control period, inference_done(latency) when a chunk arrives."""

    def __init__(self, C: int, tau_step_s: float, tau_inf_init_s: float):
        h = ctypes.c_void_p()
        _check(load().reflex_overlap_create(int(C), float(tau_step_s), float(tau_inf_init_s), ctypes.byref(h)))
        self.handle = h

    def tick(self) -> dict:
        ev = OverlapEvent()
        _check(load().reflex_overlap_tick(self.handle, ctypes.byref(ev)))
        return {n: getattr(ev, n) for n in ("chunk", "action", "launch_now", "stalled", "lookahead", "stalls_total")}

    def inference_done(self, latency_s: float):
        _check(load().reflex_overlap_inference_done(self.handle, float(latency_s)))

    def __del__(self):
        try:
            if self.handle:
                load().reflex_overlap_destroy(self.handle)
                self.handle = None
        except Exception:
            pass


def reflex_overlap_simulate(C, tau_step_s, tau_inf_init_s, tau_inf_s, mode=0, fixed_K=0) -> dict:
    arr = (ctypes.c_double * len(tau_inf_s))(*[float(t) for t in tau_inf_s])
    st = OverlapStats()
    _check(load().reflex_overlap_simulate(int(C), float(tau_step_s), float(tau_inf_init_s), arr, len(tau_inf_s), int(mode), int(fixed_K), ctypes.byref(st)))
    return {n: getattr(st, n) for n, _ in OverlapStats._fields_}
