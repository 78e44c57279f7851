"""Drives the hot path the way a serving loop would (product code: CUDA library only, no oracle).

One "denoising step" = for every layer in order: AdaRMSNorm, then partitioned attention; then the
Euler update of the action chunk. The projections that sit between those calls in the real layer are
not part of this path, so every (layer, step-variant) has its own seeded inputs resident in HBM:
all bytes the path must read are really read, and nothing is batched across layers or steps.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as rb
from . import synth


class StepRunner:
    def __init__(self, w: synth.Workload, device: str = "cuda:0", variants: int = 2, attn_impl: int = rb.ATTN_AUTO,
                 host_inputs: bool = False, ring_fill: Optional[int] = None, gate_scratch: bool = True, gate_mode: str = "tick",
                 static_banks: int = 1):
        self.w = w
        self.device = torch.device(device)
        self.variants = variants
        tdt = rb.torch_dtype(w.dtype)
        self.tdt = tdt
        g = torch.Generator(device=self.device)
        g.manual_seed(1234 + w.seed)
        self._gen = g

        def rnd(*shape, std=1.0):
            t = torch.randn(*shape, generator=g, device=self.device, dtype=torch.float32)
            if std != 1.0:
                t = t * std
            return t.to(tdt).contiguous()

        self.rnd = rnd
        head0 = [int(h) for h in synth.ring_head0(w)]
        self.cache = rb.Cache(w.L, w.B, w.Hq, w.Hkv, w.d, w.S_max, w.N, w.T, w.dtype, device=device, ring_head0=head0, static_banks=static_banks)
        rb.reflex_cache_set_attention_impl(self.cache, attn_impl)
        ids = list(range(w.B))
        # static prefix, a few streams at a time to bound the staging tensors
        chunk = max(1, min(w.B, 8))
        for i0 in range(0, w.B, chunk):
            sub = ids[i0:i0 + chunk]
            rb.reflex_cache_init_static(self.cache, sub, rnd(len(sub), w.L, w.S, w.Hkv, w.d), rnd(len(sub), w.L, w.S, w.Hkv, w.d))
        fill = w.N if ring_fill is None else ring_fill
        left = fill
        while left > 0:
            m = min(left, w.N)
            rb.reflex_cache_append_sliding(self.cache, ids, rnd(w.B, w.L, m, w.Hkv, w.d), rnd(w.B, w.L, m, w.Hkv, w.d))
            left -= m
        # per (layer, variant) inputs
        self.x = [[self._norm_input() for _ in range(variants)] for _ in range(w.L)]
        self.q = [[rnd(w.B, w.T, w.Hq, w.d) for _ in range(variants)] for _ in range(w.L)]
        self.kd = [[rnd(w.B, w.T, w.Hkv, w.d) for _ in range(variants)] for _ in range(w.L)]
        self.vd = [[rnd(w.B, w.T, w.Hkv, w.d) for _ in range(variants)] for _ in range(w.L)]
        self.vflow = [rnd(w.B, w.T, w.A) for _ in range(variants)]
        # gate-MLP parameters of all layers, stacked along a leading layer axis (self.W[l] are views of layer l)
        self.W1s, self.b1s = rnd(w.L, w.Hd, w.Cd, std=0.02), rnd(w.L, w.Hd, std=0.1)
        self.W2s, self.b2s = rnd(w.L, w.D, w.Hd, std=0.02), rnd(w.L, w.D, std=0.1)
        self.W = [[self.W1s[l], self.b1s[l], self.W2s[l], self.b2s[l]] for l in range(w.L)]
        self.cond = [torch.from_numpy(synth.cond_vectors(w, 1.0 - k / w.K)).to(self.device).to(tdt).contiguous() for k in range(w.K)]
        self.y = torch.empty((w.B, w.T, w.D), dtype=tdt, device=self.device)
        self.out = torch.empty((w.B, w.T, w.Hq, w.d), dtype=tdt, device=self.device)
        # gate [B][D] + hidden scratch [B][Hd]: lets AdaRMSNorm read the gate weights once per 16 streams
        self.gate_buf = torch.empty((w.B * (w.D + w.Hd),), dtype=torch.float32, device=self.device) if gate_scratch else None
        # The gate of Eq. 2 depends on c = [emb(t_k), s_t] only, not on any layer's input. gate_mode:
        #   "step"    (default) one call at the start of the step computes the gates of all L layers (two launches), every
        #             layer's row kernel then takes its slice as a ready gate;
        #   "overlap" the gate of layer l+1 is computed on a second stream while layer l's attention runs;
        #   "inline"  each layer's reflex_adarmsnorm call computes its own gate (three launches per layer).
        #   "tick"    one call per control tick computes the gates of all K steps and all L layers: c_k = [emb(t_k), s_t] is
        #             known for the whole schedule when the tick starts (the streams' K conditioning vectors are stacked as
        #             K * B "streams" of the gate kernels).
        self.gate_mode = gate_mode if gate_scratch else "inline"
        if gate_scratch:
            self.cond_all = torch.cat(self.cond, dim=0).contiguous()                     # [K * B][Cd]
            self.gate_tick = torch.empty((w.L * w.K * w.B * (w.D + w.Hd),), dtype=torch.float32, device=self.device)
            self.gate_all = torch.empty((w.L * w.B * (w.D + w.Hd),), dtype=torch.float32, device=self.device)
            self.gate_bufs = [torch.empty((w.B * (w.D + w.Hd),), dtype=torch.float32, device=self.device) for _ in range(2)]
            self.side = torch.cuda.Stream(device=self.device)
        self.xa = torch.randn(w.B, w.T, w.A, generator=g, device=self.device, dtype=torch.float32)
        self.host = None
        self._calls = {}
        if host_inputs:
            self._make_host_copies()
        torch.cuda.synchronize(self.device)

    def _norm_input(self):
        w = self.w
        t = torch.randn(w.B, w.T, w.D, generator=self._gen, device=self.device, dtype=torch.float32)
        if w.outlier_frac > 0:
            mask = torch.rand(w.B, w.T, w.D, generator=self._gen, device=self.device) < w.outlier_frac
            t = torch.where(mask, t * w.outlier_mult, t)
        return t.to(self.tdt).contiguous()

    # ---- bytes and flops the method must move / compute (per launch and per step) ----
    def algorithmic(self):
        w = self.w
        es = 2 if w.dtype == synth.DTYPE_BF16 else 4
        kv = (w.S + w.N + w.T) * w.Hkv * w.d * es * 2
        qo = 2 * w.T * w.Hq * w.d * es
        attn_bytes = w.B * (kv + qo)
        norm_bytes = w.B * (2 * w.T * w.D * es + w.Cd * es) + (w.Hd * w.Cd + w.D * w.Hd + w.Hd + w.D) * es
        flow_bytes = w.B * w.T * w.A * (8 + es)
        attn_flops = 4.0 * w.B * w.T * w.Hq * (w.S + w.N + w.T) * w.d
        return {"attn_bytes_per_launch": attn_bytes, "norm_bytes_per_launch": norm_bytes, "flow_bytes_per_launch": flow_bytes,
                "bytes_per_step": w.L * (attn_bytes + norm_bytes) + flow_bytes, "attn_flops_per_launch": attn_flops,
                "flops_per_step": w.L * attn_flops}

    def input_bytes_resident(self):
        n = 0
        for group in (self.x, self.q, self.kd, self.vd):
            for per_layer in group:
                for t in per_layer:
                    n += t.numel() * t.element_size()
        n += 2 * self.cache.k_slab.numel() * self.cache.k_slab.element_size()
        return n

    # ---- the step (calls are marshalled once and cached: the per-call host cost is ~1 us) ----
    def _call(self, key, make):
        c = self._calls.get(key)
        if c is None:
            c = self._calls[key] = make()
        return c

    def norm(self, layer: int, k: int, variant: int, sh=None):
        kk = k % self.w.K
        W1, b1, W2, b2 = self.W[layer]
        self._call(("n", layer, kk, variant), lambda: rb.prepare_adarmsnorm(
            self.x[layer][variant], self.y, self.cond[kk], W1, b1, W2, b2, gate_buf=self.gate_buf))(sh or rb.stream_handle())

    def attention(self, layer: int, variant: int, sh=None):
        self._call(("a", layer, variant), lambda: rb.prepare_partitioned_attention(
            self.cache, layer, self.q[layer][variant], self.kd[layer][variant], self.vd[layer][variant], self.out))(sh or rb.stream_handle())

    def flow(self, k: int, variant: int, sh=None):
        kk = k % self.w.K
        self._call(("f", kk, variant), lambda: rb.prepare_flow_step(self.xa, self.vflow[variant], None, kk, self.w.K))(sh or rb.stream_handle())

    def gate(self, layer: int, k: int, sh):
        kk = k % self.w.K
        W1, b1, W2, b2 = self.W[layer]
        self._call(("g", layer, kk), lambda: rb.prepare_adarmsnorm_gate(self.cond[kk], W1, b1, W2, b2, self.gate_bufs[layer & 1]))(sh)

    def gates_of_step(self, k: int, sh):
        """gamma_l(c_k) for all layers of this step in one call."""
        kk = k % self.w.K
        self._call(("G", kk), lambda: rb.prepare_adarmsnorm_gate(self.cond[kk], self.W1s, self.b1s, self.W2s, self.b2s, self.gate_all))(sh)

    def gates_of_tick(self, sh):
        """gamma_l(c_k) for all layers and all K steps of the tick in one call."""
        self._call(("T",), lambda: rb.prepare_adarmsnorm_gate(self.cond_all, self.W1s, self.b1s, self.W2s, self.b2s, self.gate_tick))(sh)

    def rows(self, layer: int, variant: int, sh, from_step_gates=False, k: int = 0):
        """from_step_gates: False (this layer's own gate buffer), True (gates_of_step), "tick" (gates_of_tick, step k)."""
        w = self.w
        n = w.B * w.D
        if from_step_gates == "tick":
            o = (layer * w.K + k % w.K) * n
            gate = self.gate_tick[o:o + n]
            from_step_gates = ("tick", k % w.K)
        else:
            gate = self.gate_all[layer * n:(layer + 1) * n] if from_step_gates else self.gate_bufs[layer & 1][:n]
        self._call(("r", layer, variant, from_step_gates), lambda: rb.prepare_adarmsnorm(
            self.x[layer][variant], self.y, None, None, None, None, None, gate_buf=gate.view(w.B, w.D)))(sh)

    # ---- chained layer: the norm output feeds the packed Q/K/V projection, whose output feeds attention ----
    def _chained_buffers(self):
        if not hasattr(self, "Wqkv"):
            w = self.w
            self.Wqkv = [self.rnd((w.Hq + 2 * w.Hkv) * w.d, w.D, std=float(w.D) ** -0.5) for _ in range(w.L)]
            self.qc = torch.empty((w.B, w.T, w.Hq, w.d), dtype=self.tdt, device=self.device)
            self.kc = torch.empty((w.B, w.T, w.Hkv, w.d), dtype=self.tdt, device=self.device)
            self.vc = torch.empty((w.B, w.T, w.Hkv, w.d), dtype=self.tdt, device=self.device)

    def norm_qkv(self, layer: int, variant: int, sh, impl: int = 0):
        """AdaRMSNorm folded into the packed projection: x_l -> Q, K_dyn, V_dyn (gates from gates_of_step)."""
        self._chained_buffers()
        w = self.w
        n = w.B * w.D
        gate = self.gate_all[layer * n:(layer + 1) * n].view(w.B, w.D)
        self._call(("q", layer, variant, impl), lambda: rb.prepare_adarmsnorm_qkv(
            self.x[layer][variant], gate, self.Wqkv[layer], self.qc, self.kc, self.vc, impl=impl, cache=self.cache))(sh)

    def norm_swiglu(self, layer: int, variant: int, sh, F: Optional[int] = None):
        """AdaRMSNorm folded into the fused gate / up projections of the layer's SwiGLU block: x_l -> h [B][T][F]."""
        w = self.w
        F = 4 * w.D if F is None else F
        if not hasattr(self, "Wgu") or self.Wgu[0].shape[0] != 2 * F:
            self.Wgu = [self.rnd(2 * F, w.D, std=float(w.D) ** -0.5) for _ in range(w.L)]
            self.hmlp = torch.empty((w.B, w.T, F), dtype=self.tdt, device=self.device)
        n = w.B * w.D
        gate = self.gate_all[layer * n:(layer + 1) * n].view(w.B, w.D)
        self._call(("s", layer, variant, F), lambda: rb.prepare_adarmsnorm_swiglu(
            self.x[layer][variant], gate, self.Wgu[layer], self.hmlp, cache=self.cache))(sh)

    def attention_chained(self, layer: int, sh):
        self._chained_buffers()
        self._call(("ac", layer), lambda: rb.prepare_partitioned_attention(self.cache, layer, self.qc, self.kc, self.vc, self.out))(sh)

    def step_chained(self, k: int):
        """A denoising step in which every layer's norm + Q/K/V projection produces the tensors its attention reads."""
        variant = k % self.variants
        sh = rb.stream_handle(torch.cuda.current_stream())
        self.gates_of_step(k, sh)
        for layer in range(self.w.L):
            self.norm_qkv(layer, variant, sh)
            self.attention_chained(layer, sh)
        self.flow(k, variant, sh)

    def step(self, k: int):
        """One denoising step over all layers and streams, inputs already in HBM."""
        variant = k % self.variants
        main = torch.cuda.current_stream()
        sh = rb.stream_handle(main)
        if self.gate_mode == "tick":
            if k % self.w.K == 0:
                self.gates_of_tick(sh)
            for layer in range(self.w.L):
                self.rows(layer, variant, sh, "tick", k)
                self.attention(layer, variant, sh)
        elif self.gate_mode == "step":
            self.gates_of_step(k, sh)
            for layer in range(self.w.L):
                self.rows(layer, variant, sh, True)
                self.attention(layer, variant, sh)
        elif self.gate_mode == "overlap":
            side_h = rb.stream_handle(self.side)
            self.gate(0, k, sh)
            for layer in range(self.w.L):
                self.rows(layer, variant, sh)
                if layer + 1 < self.w.L:
                    self.side.wait_stream(main)          # the next gate may start once this layer's rows are queued
                    self.gate(layer + 1, k, side_h)
                self.attention(layer, variant, sh)
                if layer + 1 < self.w.L:
                    main.wait_stream(self.side)          # ... and must be complete before the next layer's rows
        else:
            for layer in range(self.w.L):
                self.norm(layer, k, variant, sh)
                self.attention(layer, variant, sh)
        self.flow(k, variant, sh)

    # ---- CUDA graphs: the launch-bound inner loop is captured once and replayed (host cost per step: one launch) ----
    def capture(self, fn):
        """Capture the library calls made by fn() into a CUDA graph; returns (graph, number of kernels in it)."""
        fn()                                   # warm-up outside capture (first-call set-up, lazy module loading)
        torch.cuda.synchronize(self.device)
        g = torch.cuda.CUDAGraph()
        n0 = rb.reflex_kernel_launch_count()
        with torch.cuda.graph(g):
            fn()
        return g, rb.reflex_kernel_launch_count() - n0

    def capture_steps(self):
        """One graph per distinct step (conditioning index x input variant)."""
        import math
        period = self.w.K * self.variants // math.gcd(self.w.K, self.variants)
        self.step_graphs, self.kernels_per_step, self.kernels_each = [], 0, []
        for k in range(period):
            g, n = self.capture(lambda k=k: self.step(k))
            self.step_graphs.append(g)
            self.kernels_each.append(n)
            self.kernels_per_step = n
        return self.step_graphs

    # ---- one control tick of the stream: ring append, fresh noise, K denoising steps ----
    def tick(self):
        w = self.w
        sh = rb.stream_handle()
        if not hasattr(self, "_tick_src"):
            self._tick_src = (self.rnd(w.B, w.L, w.m, w.Hkv, w.d), self.rnd(w.B, w.L, w.m, w.Hkv, w.d),
                              torch.randn(w.B, w.T, w.A, generator=self._gen, device=self.device, dtype=torch.float32))
            self._ids = list(range(w.B))
        kn, vn, noise = self._tick_src
        rb.reflex_cache_append_sliding(self.cache, self._ids, kn, vn)      # O(m) in-place append in every layer
        self.xa.copy_(noise)                                               # x ~ N(0, I) at t = 1
        for k in range(w.K):
            self.step(k)

    def capture_tick(self):
        self.tick_graph, self.kernels_per_tick = self.capture(self.tick)
        return self.tick_graph

    def refresh_static(self, S: int):
        """A new observation: rewrite the static prefix of every stream (S tokens), as happens every few ticks."""
        w = self.w
        if not hasattr(self, "_static_src"):
            self._static_src = (self.rnd(w.B, w.L, w.S_max, w.Hkv, w.d), self.rnd(w.B, w.L, w.S_max, w.Hkv, w.d))
        ks, vs = self._static_src
        rb.reflex_cache_init_static(self.cache, list(range(w.B)), ks, vs, S=[S] * w.B)

    def stage_static(self, S: int, stream):
        """Producer side of the asynchronous pipeline: the next observation's prefix goes to the idle static bank on
        `stream` while the denoising steps keep reading the current one (cache created with static_banks=2)."""
        w = self.w
        if not hasattr(self, "_static_src"):
            self._static_src = (self.rnd(w.B, w.L, w.S_max, w.Hkv, w.d), self.rnd(w.B, w.L, w.S_max, w.Hkv, w.d))
        ks, vs = self._static_src
        rb.reflex_cache_stage_static(self.cache, list(range(w.B)), ks, vs, S=[S] * w.B, stream=stream)

    def commit_static(self):
        """Consumer side, between two ticks: the staged prefix becomes the current one (index flip)."""
        rb.reflex_cache_commit_static(self.cache, list(range(self.w.B)))

    def step_graph(self, k: int):
        self.step_graphs[k % len(self.step_graphs)].replay()

    def step_timed(self, k: int, ev_attn, ev_norm):
        """Same launches as step(), with CUDA events around every attention and norm call."""
        variant = k % self.variants
        rec = lambda: (lambda e: (e.record(), e)[1])(torch.cuda.Event(enable_timing=True))
        for layer in range(self.w.L):
            a = rec(); self.norm(layer, k, variant); b = rec(); self.attention(layer, variant); c = rec()
            ev_norm.append((a, b)); ev_attn.append((b, c))
        self.flow(k, variant)

    # ---- end to end: this step's inputs come from pinned host memory, the action chunk goes back ----
    def _make_host_copies(self):
        pin = lambda t: t.cpu().pin_memory()
        self.host = {name: [[pin(t) for t in per_layer] for per_layer in getattr(self, name)] for name in ("x", "q", "kd", "vd")}
        self.host["vflow"] = [pin(t) for t in self.vflow]
        self.host_xa = torch.empty(self.xa.shape, dtype=torch.float32).pin_memory()
        nb = lambda t: t.numel() * t.element_size()
        self.h2d_bytes_per_step = sum(nb(self.host[n][l][0]) for n in ("x", "q", "kd", "vd") for l in range(self.w.L)) + nb(self.host["vflow"][0])
        self.d2h_bytes_per_step = nb(self.host_xa)

    def copy_inputs_from_host(self, k: int):
        """This step's inputs (every layer's x, Q, K_dyn, V_dyn and the velocity) from pinned host memory."""
        variant = k % self.variants
        for layer in range(self.w.L):
            for name in ("x", "q", "kd", "vd"):
                getattr(self, name)[layer][variant].copy_(self.host[name][layer][variant], non_blocking=True)
        self.vflow[variant].copy_(self.host["vflow"][variant], non_blocking=True)

    def copy_result_to_host(self):
        self.host_xa.copy_(self.xa, non_blocking=True)
