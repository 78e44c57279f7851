"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element on the
same seeded inputs. Integer / byte work is compared exactly, floating point within the contract
tolerances (bf16: max-abs 2e-2, mean-abs 2e-3 against the fp64 oracle; fp32 storage: 2e-5 / 2e-6)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2607_14695_b200 import synth  # noqa: E402


@pytest.fixture(scope="module")
def U():
    from paper_2607_14695_b200 import build as rbuild
    rbuild.build()
    import gpu_util
    return gpu_util


def _gate_tol(orc, cond_b, W1, b1, W2, b2):
    """Bound on the fp32 gate against the double-precision one: fp32 accumulation (1e-5 at gates of order 1) plus, on the
    tensor-core path, the hidden activations passed on as two bf16 halves (relative 2^-16 each, weighted by |W2|)."""
    z = W1.astype(np.float64) @ cond_b.astype(np.float64) + b1
    h = np.abs(z / (1.0 + np.exp(-z)))
    return 1e-5 + 2.0 ** -16 * (np.abs(W2).astype(np.float64) @ h)


def _norm_case(U, w, x, cond, layer=0, eps=1e-6, gate_buf=False, alias=False, what="adarmsnorm", std=0.02, bias_std=0.1):
    from oracle import reflex_oracle as orc
    rb = U.rb
    W1, b1, W2, b2 = synth.gate_weights(w, layer, std=std, bias_std=bias_std)
    dx = U.to_dev(x, w.dtype)
    dy = dx if alias else torch.full_like(dx, float("nan"))
    gb = torch.empty((x.shape[0] * (w.D + w.Hd),), dtype=torch.float32, device=U.DEV) if gate_buf else None
    rb.reflex_adarmsnorm(dx, dy, U.to_dev(cond, w.dtype), U.to_dev(W1, w.dtype), U.to_dev(b1, w.dtype), U.to_dev(W2, w.dtype),
                         U.to_dev(b2, w.dtype), gate_buf=gb, eps=eps)
    want = orc.adarmsnorm_batched(x, cond, W1, b1, W2, b2, eps)
    U.check_close(U.to_host(dy), want, w.dtype, what, rel_clause=True)
    if gate_buf:  # the gate itself, fp32, and the precomputed-gate entry
        for b in sorted({0, x.shape[0] - 1}):
            _, g0 = orc.adarmsnorm(x[b], cond[b], W1, b1, W2, b2, eps, return_gate=True)
            assert (np.abs(U.to_host(gb[b * w.D:(b + 1) * w.D]) - g0) <= _gate_tol(orc, cond[b], W1, b1, W2, b2)).all(), what + ": gate"
        dy2 = torch.full_like(dx, float("nan"))
        rb.reflex_adarmsnorm(U.to_dev(x, w.dtype), dy2, None, None, None, None, None, gate_buf=gb[: x.shape[0] * w.D].view(x.shape[0], w.D), eps=eps)
        assert torch.equal(dy2, dy)
    return dy


# ------------------------------------------------------------------------------------------------
# config 1: tiny fp32 layer, 40 ticks x 4 Euler steps, every call of every tick compared
# ------------------------------------------------------------------------------------------------
def test_cfg1_full_trace(U):
    from oracle import reflex_oracle as orc
    rb = U.rb
    w = synth.CONFIGS["cfg1"]
    tw = U.Twin(w)
    tw.init_static([0], [w.S])
    W1, b1, W2, b2 = synth.gate_weights(w, 0, std=0.2)
    dW = [U.to_dev(a, w.dtype) for a in (W1, b1, W2, b2)]
    evicted_total = 0
    for tick in range(w.ticks):
        evicted_total += tw.append([0], 1, tick)[0]
        tw.check_state()
        assert tw.o.head[0] == (tick + 1) % 16 and tw.o.count[0] == min(tick + 1, 16)
        x0 = synth.normal(w, "noise", (w.B, w.T, w.A), 0, tick)
        x_or = x0.astype(np.float64).copy()
        x_gpu = torch.from_numpy(x0).to(U.DEV)
        for k in range(w.K):
            variant = tick * w.K + k
            t_k = orc.flow_time(k, w.K)
            # norm -> attention chained literally: D = Hq*d = 128, so Q = y viewed [T][2][64], K_d = y[:, :64], V_d = y[:, 64:]
            x = synth.normal(w, "x", (w.B, w.T, w.D), 0, variant)
            cond = synth.cond_vectors(w, t_k, variant=tick)
            dy = torch.empty((w.B, w.T, w.D), dtype=torch.float32, device=U.DEV)
            rb.reflex_adarmsnorm(U.to_dev(x, w.dtype), dy, U.to_dev(cond, w.dtype), *dW, eps=1e-6)
            y_or = orc.adarmsnorm_batched(x, cond, W1, b1, W2, b2, 1e-6)
            U.check_close(U.to_host(dy), y_or, w.dtype, f"norm tick {tick} step {k}", rel_clause=True)
            y32 = dy.cpu().numpy()   # the oracle continues from the GPU's fp32 y so errors do not compound across calls
            q = y32.reshape(w.B, w.T, w.Hq, w.d)
            kd = np.ascontiguousarray(y32[:, :, :64]).reshape(w.B, w.T, 1, 64)
            vd = np.ascontiguousarray(y32[:, :, 64:]).reshape(w.B, w.T, 1, 64)
            out = torch.empty((w.B, w.T, w.Hq, w.d), dtype=torch.float32, device=U.DEV)
            rb.reflex_partitioned_attention(tw.g, 0, dy.view(w.B, w.T, w.Hq, w.d), U.to_dev(kd, w.dtype), U.to_dev(vd, w.dtype), out)
            want = tw.o.attention(0, 0, q[0], kd[0], vd[0])
            U.check_close(U.to_host(out)[0], want, w.dtype, f"attention tick {tick} step {k}")
            v = synth.normal(w, "v_flow", (w.B, w.T, w.A), 0, variant)
            rb.reflex_flow_step(x_gpu, U.to_dev(v, w.dtype), None, k, w.K)
            orc.flow_step(x_or, v, w.K)
        U.check_close(U.to_host(x_gpu), x_or, w.dtype, f"action chunk tick {tick}")
    assert evicted_total == 24


# ------------------------------------------------------------------------------------------------
# config 2: one pi0-class layer, batch 1, bf16
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", ["simt", "tc", "tc2"])
@pytest.mark.parametrize("count", [5, 32, 45])
def test_cfg2_layer(U, impl, count):
    rb = U.rb
    w = synth.CONFIGS["cfg2"]
    tw = U.Twin(w, head0=[7], poison=True)
    rb.reflex_cache_set_attention_impl(tw.g, {"simt": rb.ATTN_SIMT, "tc": rb.ATTN_TC, "tc2": rb.ATTN_TC2}[impl])
    tw.init_static([0], [w.S])
    for i in range(count):
        tw.append([0], 1, i)
    tw.check_state()
    for dyn_mask in (0, 1):
        tw.attention(0, 10 + dyn_mask, dyn_mask=dyn_mask, what=f"cfg2 attention mask={dyn_mask}")
        tw.attention(0, 10 + dyn_mask, dyn_mask=dyn_mask, partitioned=True, what="cfg2 attention vs partitioned oracle")
    tw.check_state()   # attention only reads the cached regions (timestep invariance)
    # AdaRMSNorm over the 10-step schedule and the Euler chain
    from oracle import reflex_oracle as orc
    for k in (0, 3, 9):
        x = synth.norm_input(w, 0, k)
        cond = synth.cond_vectors(w, orc.flow_time(k, w.K))
        _norm_case(U, w, x, cond, gate_buf=(k == 3), alias=(k == 9), what=f"cfg2 norm step {k}")
    x0 = synth.normal(w, "noise", (w.B, w.T, w.A))
    x_or = x0.astype(np.float64).copy(); x_gpu = torch.from_numpy(x0).to(U.DEV)
    mirror = torch.empty((w.B, w.T, w.A), dtype=torch.bfloat16, device=U.DEV)
    for k in range(w.K):
        v = synth.normal(w, "v_flow", (w.B, w.T, w.A), 0, k)
        rb.reflex_flow_step(x_gpu, U.to_dev(v, w.dtype), mirror, k, w.K)
        orc.flow_step(x_or, v, w.K)
    U.check_close(U.to_host(x_gpu), x_or, synth.DTYPE_F32, "cfg2 action chunk (fp32 master)")
    assert torch.equal(mirror, x_gpu.to(torch.bfloat16))


# ------------------------------------------------------------------------------------------------
# config 3 shapes: 18 layers, streaming ticks with a new (shorter) prefix, stale rows poisoned
# ------------------------------------------------------------------------------------------------
def test_cfg3_stream_ticks(U):
    w = synth.CONFIGS["cfg3"]
    tw = U.Twin(w, head0=[30], poison=True)
    S_sched = {0: 816, 10: 800, 20: 816}
    for tick in range(0, 34):
        if tick in S_sched:
            tw.init_static([0], [S_sched[tick]], variant=tick)
        tw.append([0], 1, tick)
        if tick in (0, 1, 9, 10, 11, 31, 32, 33):
            tw.check_state()
            for layer in ((0, 17) if tick not in (10, 32) else range(w.L)):
                tw.attention(layer, tick, what=f"cfg3 tick {tick}")


def test_cfg3_500_tick_stream_graph_replay(U):
    """The batch-1 streaming trace in full: 500 control ticks, one token appended to the ring in all 18 layers per tick, a
    new static prefix every 10 ticks with lengths alternating 816 / 800 (a shorter prefix leaves stale rows behind). From
    tick 1 on a tick is ONE CUDA-graph replay (ring append + 18 attention launches) fed through fixed device buffers; the
    oracle is advanced on the host with the same bytes. Ring state, slot map and cache bytes are compared exactly and the
    attention outputs element-wise on ticks 0, 1, 9, 10, 11, 31, 32, 33 and 499 (the ring has wrapped 15 times by then)."""
    rb = U.rb
    w = synth.CONFIGS["cfg3"]
    tw = U.Twin(w, head0=[30], poison=True)
    dt = rb.torch_dtype(w.dtype)
    e = lambda *s: torch.empty(s, dtype=dt, device=U.DEV)
    kn_buf, vn_buf = e(1, w.L, 1, w.Hkv, w.d), e(1, w.L, 1, w.Hkv, w.d)
    q_buf, kd_buf, vd_buf = e(w.L, 1, w.T, w.Hq, w.d), e(w.L, 1, w.T, w.Hkv, w.d), e(w.L, 1, w.T, w.Hkv, w.d)
    out_buf = e(w.L, 1, w.T, w.Hq, w.d)

    def tick_calls():
        rb.reflex_cache_append_sliding(tw.g, [0], kn_buf, vn_buf)
        for layer in range(w.L):
            rb.reflex_partitioned_attention(tw.g, layer, q_buf[layer], kd_buf[layer], vd_buf[layer], out_buf[layer])

    def fill_inputs(tick):
        host = {}
        for layer in range(w.L):
            host[layer] = tuple(synth.normal(w, n, (1, w.T, h, w.d), layer, tick) for n, h in (("q", w.Hq), ("k_dyn", w.Hkv), ("v_dyn", w.Hkv)))
            for buf, a in zip((q_buf, kd_buf, vd_buf), host[layer]):
                buf[layer].copy_(U.to_dev(a, w.dtype))
        return host

    compare = {0, 1, 9, 10, 11, 31, 32, 33, 499}
    graph = None
    fill_inputs(0)
    for tick in range(500):
        if tick % 10 == 0:
            tw.init_static([0], [816 if (tick // 10) % 2 == 0 else 800], variant=tick)
        kn = synth.normal(w, "k_new", (1, w.L, 1, w.Hkv, w.d), 0, tick)
        vn = synth.normal(w, "v_new", (1, w.L, 1, w.Hkv, w.d), 0, tick)
        tw.o.append_sliding(0, kn[0], vn[0])
        kn_buf.copy_(U.to_dev(kn, w.dtype)); vn_buf.copy_(U.to_dev(vn, w.dtype))
        host = fill_inputs(tick) if tick in compare else None
        if tick == 0:
            tick_calls()                       # direct launches; the graph is captured afterwards (capture launches nothing)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                tick_calls()
        else:
            graph.replay()
        if tick in compare:
            torch.cuda.synchronize()
            rb.reflex_cache_check_status(tw.g)
            tw.check_state()                   # (reads the ring state back from the device: replays do not touch the host mirror)
            assert tw.o.total[0] == tick + 1 and tw.o.count[0] == min(tick + 1, w.N) and tw.o.head[0] == (30 + tick + 1) % w.N
            got = U.to_host(out_buf)
            assert np.isfinite(got).all()
            for layer in (range(w.L) if tick in (10, 32, 499) else (0, 17)):
                q, kd, vd = host[layer]
                want = tw.o.attention(0, layer, q[0], kd[0], vd[0])
                U.check_close(got[layer, 0], want, w.dtype, f"cfg3 tick {tick} layer {layer}")


# ------------------------------------------------------------------------------------------------
# config 4 shapes: 64 streams with random ring offsets and mixed fill levels
# ------------------------------------------------------------------------------------------------
def test_cfg4_batched_streams(U):
    w = synth.CONFIGS["cfg4"].with_(L=3)
    head0 = synth.ring_head0(w)
    tw = U.Twin(w, head0=head0, poison=True)
    tw.init_static(list(range(w.B)), [w.S] * w.B)
    # 60 streams get >= 32 appends (full rings at different offsets), 4 stay partially filled
    for i in range(40):
        ids = [b for b in range(w.B) if not (b in (5, 17, 40, 63) and i >= 3 + b % 7)]
        tw.append(ids, 1, i)
    tw.check_state()
    assert sorted(set(tw.o.count)) != [32]
    tw.attention(0, 0, streams=[0, 5, 17, 31, 40, 62, 63], what="cfg4 step 0")
    tw.attention(2, 9, streams=[1, 63], what="cfg4 step 9")
    from oracle import reflex_oracle as orc
    x = synth.norm_input(w, 1, 0)
    _norm_case(U, w, x, synth.cond_vectors(w, 0.7), layer=1, what="cfg4 norm")
    _norm_case(U, w, x, synth.cond_vectors(w, 0.2), layer=1, gate_buf=True, what="cfg4 norm two-launch")


# ------------------------------------------------------------------------------------------------
# config 5 shapes: long context, outliers in the norm input, t near 0 and 1
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", ["auto", "tc2"])
def test_cfg5_long_context(U, impl):
    w = synth.CONFIGS["cfg5"].with_(L=2, B=4)
    tw = U.Twin(w, head0=synth.ring_head0(w), poison=True)
    U.rb.reflex_cache_set_attention_impl(tw.g, U.rb.ATTN_AUTO if impl == "auto" else U.rb.ATTN_TC2)
    tw.init_static(list(range(w.B)), [w.S, w.S - 100, w.S, 1])
    for i in range(3):
        tw.append(list(range(w.B)), 100, i)      # frame-sized appends; wraps the 256-slot ring
    tw.check_state()
    tw.attention(1, 0, streams=[0, 1, 3], what="cfg5 attention")
    for t in (0.0, 1e-4, 1e-3, 1 - 1e-3, 1 - 1e-4, 1.0):
        x = synth.norm_input(w, 0, int(t * 1000))
        assert (np.abs(x) > 100).any()
        _norm_case(U, w, x, synth.cond_vectors(w, t), what=f"cfg5 norm t={t}")


def test_cfg5b_outliers_in_queries_and_keys(U):
    """The labelled stress run beside the long-context configuration: 0.1 % of the elements of Q, of the dynamic K and of the
    cached K (prefix and ring) are multiplied by 1000, V stays N(0, 1). Logits reach tens of thousands and the softmax is
    one-hot for the rows an outlier touches: every output must be finite, and the outputs are compared with the oracle
    under the output-spacing clause (a one-hot row returns a single V row, |v| up to 4.5). This is a finiteness and
    relative-error stress outside the absolute-error contract; the worst relative error is printed."""
    rb = U.rb
    w = synth.CONFIGS["cfg5"].with_(L=1, B=3)
    tw = U.Twin(w, head0=synth.ring_head0(w), poison=True)

    def spiked(name, shape, layer, variant):
        a = synth.normal(w, name, shape, layer, variant)
        mask = synth.rng_for(w, "outlier_mask", layer, variant + 100 * synth.TID[name]).random(size=a.shape) < w.outlier_frac
        return synth.round_storage(np.where(mask, a * np.float32(w.outlier_mult), a).astype(np.float32), w.dtype)

    ids = list(range(w.B))
    ks, vs = spiked("k_static", (w.B, w.L, w.S, w.Hkv, w.d), 0, 0), synth.normal(w, "v_static", (w.B, w.L, w.S, w.Hkv, w.d), 0, 0)
    for b in ids:
        tw.o.init_static(b, ks[b], vs[b])
    rb.reflex_cache_init_static(tw.g, ids, U.to_dev(ks, w.dtype), U.to_dev(vs, w.dtype))
    for i in range(3):
        kn, vn = spiked("k_new", (w.B, w.L, 100, w.Hkv, w.d), 0, i), synth.normal(w, "v_new", (w.B, w.L, 100, w.Hkv, w.d), 0, i)
        for b in ids:
            tw.o.append_sliding(b, kn[b], vn[b])
        rb.reflex_cache_append_sliding(tw.g, ids, U.to_dev(kn, w.dtype), U.to_dev(vn, w.dtype))
    tw.check_state()
    q, kd = spiked("q", (w.B, w.T, w.Hq, w.d), 0, 0), spiked("k_dyn", (w.B, w.T, w.Hkv, w.d), 0, 0)
    vd = synth.normal(w, "v_dyn", (w.B, w.T, w.Hkv, w.d), 0, 0)
    assert (np.abs(q) > 100).any() and (np.abs(ks) > 100).any() and (np.abs(kd) > 100).any()
    worst_rel = 0.0
    for impl in (rb.ATTN_AUTO, rb.ATTN_TC, rb.ATTN_SIMT):
        rb.reflex_cache_set_attention_impl(tw.g, impl)
        for dyn_mask in (0, 1):
            out = torch.full((w.B, w.T, w.Hq, w.d), float("nan"), dtype=torch.bfloat16, device=U.DEV)
            rb.reflex_partitioned_attention(tw.g, 0, U.to_dev(q, w.dtype), U.to_dev(kd, w.dtype), U.to_dev(vd, w.dtype), out, dyn_mask=dyn_mask)
            rb.reflex_cache_check_status(tw.g)
            got = U.to_host(out)
            assert np.isfinite(got).all(), "cfg5b: non-finite output"
            for b in ids:
                want = tw.o.attention(b, 0, q[b], kd[b], vd[b], dyn_mask, None)
                U.check_close(got[b], want, w.dtype, f"cfg5b stream {b} mask {dyn_mask} impl {impl}", rel_clause=True)
                big = np.abs(want) > 0.5
                if big.any():
                    worst_rel = max(worst_rel, float((np.abs(got[b] - want)[big] / np.abs(want)[big]).max()))
    print(f"cfg5b: worst relative error on |o| > 0.5: {worst_rel:.3e}")
    assert worst_rel <= U.BF16_MAX_ABS / 0.5          # (what the element-wise bound above allows at |o| = 0.5)


# ------------------------------------------------------------------------------------------------
# edge cases and degenerate shapes
# ------------------------------------------------------------------------------------------------
EDGE = [
    # name, B, L, Hq, Hkv, d, S_max, S, N, T, appends(m list), dtype
    ("S0_T1_N1", 2, 1, 2, 2, 32, 4, 0, 1, 1, [1, 1], synth.DTYPE_F32),
    ("gqa4to2_d64", 3, 2, 4, 2, 64, 40, 33, 5, 7, [2, 2, 2], synth.DTYPE_BF16),
    ("mha_d128", 1, 1, 3, 3, 128, 70, 70, 9, 33, [9, 4], synth.DTYPE_BF16),
    ("m_equals_N", 2, 1, 8, 1, 256, 100, 64, 16, 17, [16, 16, 3], synth.DTYPE_BF16),
    ("empty_ring", 1, 1, 8, 1, 256, 130, 129, 8, 50, [], synth.DTYPE_BF16),
    ("f32_d256", 1, 1, 8, 2, 256, 65, 65, 33, 5, [33, 1], synth.DTYPE_F32),
    ("long_dyn_T130", 2, 1, 8, 1, 256, 200, 191, 70, 130, [70, 5], synth.DTYPE_BF16),       # several dynamic and ring tiles
    ("g16_two_kv", 2, 2, 32, 2, 128, 96, 64, 64, 9, [64], synth.DTYPE_BF16),               # G = 16, exact tile boundaries
    ("g3_simt_only", 1, 1, 6, 2, 64, 20, 20, 4, 5, [3], synth.DTYPE_BF16),                 # 128 % G != 0: SIMT even on auto
]


@pytest.mark.parametrize("impl", ["simt", "auto", "tc2"])
@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
def test_edge_shapes(U, case, impl):
    name, B, L, Hq, Hkv, d, S_max, S, N, T, appends, dtype = case
    w = synth.Workload(name, 77, dtype, B=B, L=L, Hq=Hq, Hkv=Hkv, d=d, S=S, S_max=S_max, N=N, T=T, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w, head0=[(3 * b) % N for b in range(B)], T_max=T + 3, poison=True)
    U.rb.reflex_cache_set_attention_impl(tw.g, {"simt": U.rb.ATTN_SIMT, "auto": U.rb.ATTN_AUTO, "tc2": U.rb.ATTN_TC2}[impl])
    if impl == "tc2" and not (dtype == synth.DTYPE_BF16 and d in (128, 256) and 128 % (Hq // Hkv) == 0):
        tw.init_static(list(range(B)), [S] * B)
        z = torch.zeros((B, T, Hq, d), dtype=U.rb.torch_dtype(dtype), device=U.DEV)
        zk = torch.zeros((B, T, Hkv, d), dtype=U.rb.torch_dtype(dtype), device=U.DEV)
        with pytest.raises(U.rb.ReflexError) as e:       # the two-CTA kernel refuses shapes it cannot run; nothing is launched
            U.rb.reflex_partitioned_attention(tw.g, 0, z, zk, zk, z)
        assert e.value.code == U.rb.ERR_NOT_IMPLEMENTED
        return
    tw.init_static(list(range(B)), [S] * B)
    for i, m in enumerate(appends):
        tw.append(list(range(B)), m, i)
    tw.check_state()
    for layer in range(L):
        for dyn_mask in (0, 1):
            tw.attention(layer, dyn_mask, dyn_mask=dyn_mask, what=name)
    if T > 1:
        tw.attention(0, 5, T=T - 1, what=name + " T<T_max")
    tw.attention(0, 6, scale=0.05, what=name + " scale override")


def _random_attention_cases(n, seed):
    """Seeded shapes across what the kernels branch on: head_dim, queries per KV head, KV heads, prefix lengths that differ per
    stream (0 included), ring capacity and fill (empty, partly filled, wrapped), dynamic tokens from 1 to beyond one tile."""
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        d = int(rng.choice([64, 128, 256]))
        G = int(rng.choice([1, 2, 4, 8, 16]))
        Hkv = int(rng.choice([1, 2]))
        B = int(rng.integers(1, 5))
        S_max = int(rng.choice([8, 70, 130, 300, 600]))
        N = int(rng.choice([1, 7, 32, 64, 100, 200]))
        T = int(rng.choice([1, 3, 17, 50, 64, 65, 140]))
        S_list = [int(rng.integers(0, S_max + 1)) for _ in range(B)]
        if i % 4 == 0:
            S_list[0] = S_max
        n_app = int(rng.integers(0, 4))
        appends = [int(rng.integers(1, N + 1)) for _ in range(n_app)]
        head0 = [int(rng.integers(0, N)) for _ in range(B)]
        cases.append((f"r{i}_d{d}_g{G}_kv{Hkv}_B{B}_S{S_max}_N{N}_T{T}", d, G, Hkv, B, S_max, N, T, S_list, appends, head0))
    return cases


RANDOM_CASES = _random_attention_cases(20, 2607)


@pytest.mark.parametrize("case", RANDOM_CASES, ids=[c[0] for c in RANDOM_CASES])
def test_random_shapes_every_attention_kernel(U, case):
    """Each seeded shape through every attention kernel that takes it (plain, one-CTA and two-CTA tensor-core forms, and the
    library's own choice), both masks, against the oracle element by element; ring state and cache bytes exactly."""
    name, d, G, Hkv, B, S_max, N, T, S_list, appends, head0 = case
    rb = U.rb
    w = synth.Workload(name, 99, synth.DTYPE_BF16, B=B, L=1, Hq=G * Hkv, Hkv=Hkv, d=d, S=S_max, S_max=S_max, N=N, T=T, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w, head0=head0, poison=True)
    tw.init_static(list(range(B)), S_list)
    for i, m in enumerate(appends):
        tw.append(list(range(B)), m, i)
    tw.check_state()
    tensor_core = d in (64, 128, 256) and 128 % G == 0
    two_cta = tensor_core and d in (128, 256)
    impls = [("auto", rb.ATTN_AUTO), ("simt", rb.ATTN_SIMT)] + ([("tc", rb.ATTN_TC)] if tensor_core else []) + ([("tc2", rb.ATTN_TC2)] if two_cta else [])
    for iname, impl in impls:
        rb.reflex_cache_set_attention_impl(tw.g, impl)
        for dyn_mask in (0, 1):
            tw.attention(0, dyn_mask, dyn_mask=dyn_mask, what=f"{name} {iname} mask {dyn_mask}")


@pytest.mark.parametrize("impl", ["tc", "tc2"])
def test_wide_logits_exercise_the_lazy_rescale(U, impl):
    """Queries scaled up so that row maxima keep growing by more than 2^8 from tile to tile: O and l are rescaled in
    tensor memory over and over, with and without the causal mask over the dynamic tokens. With logits this wide a row's
    output is close to single V rows (|v| up to 4.5), where the bf16 spacing of the output itself passes 2e-2: the bf16
    output-spacing allowance applies."""
    w = synth.Workload("wide", 31, synth.DTYPE_BF16, B=3, L=1, Hq=8, Hkv=1, d=256, S=700, S_max=704, N=40, T=50, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w, head0=[5, 0, 39], poison=True)
    U.rb.reflex_cache_set_attention_impl(tw.g, {"tc": U.rb.ATTN_TC, "tc2": U.rb.ATTN_TC2}[impl])
    tw.init_static(list(range(w.B)), [700, 650, 1])
    for i in range(3):
        tw.append(list(range(w.B)), 17, i)
    for q_scale in (6.0, 20.0):
        tw.attention(0, 1, dyn_mask=0, q_scale=q_scale, rel_clause=True, what=f"wide logits x{q_scale} {impl}")
        tw.attention(0, 2, dyn_mask=1, q_scale=q_scale, rel_clause=True, what=f"wide logits x{q_scale} causal {impl}")


def test_two_cta_kernel_many_units_head_dim_128(U):
    """More work units than SM pairs at head_dim 128 (four K and four V stages), two KV heads, several key tiles per unit:
    the persistent loop crosses unit boundaries with every stage and buffer rotation."""
    w = synth.Workload("units128", 32, synth.DTYPE_BF16, B=42, L=1, Hq=8, Hkv=2, d=128, S=300, S_max=320, N=48, T=20, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w, head0=[(7 * b) % w.N for b in range(w.B)], poison=True)
    U.rb.reflex_cache_set_attention_impl(tw.g, U.rb.ATTN_TC2)
    tw.init_static(list(range(w.B)), [300 - (b % 5) * 31 for b in range(w.B)])
    for i in range(4):
        tw.append([b for b in range(w.B) if not (b % 9 == 4 and i >= 2)], 16, i)
    tw.check_state()
    tw.attention(0, 0, dyn_mask=0, what="units128")
    tw.attention(0, 1, dyn_mask=1, streams=[0, 4, 13, 41], what="units128 causal")


@pytest.mark.parametrize("T", [25, 100])
def test_frame_granular_window(U, T):
    """The ablation shapes of the paper's context-window study: a sliding window of 10 frames x 256 tokens fed one frame
    (m = 256) per tick, action chunks of 25 and 100 tokens. The ring wraps several times at different offsets per stream."""
    w = synth.Workload("frames", 41, synth.DTYPE_BF16, B=3, L=1, Hq=8, Hkv=1, d=256, S=300, S_max=320, N=2560, T=T, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w, head0=[0, 1000, 2559], poison=True)
    tw.init_static(list(range(w.B)), [300, 257, 64])
    for i in range(13):                      # 13 frames into a 10-frame window; stream 2 joins late and stays partly filled
        tw.append([b for b in range(w.B) if not (b == 2 and i < 6)], 256, i)
        if i in (2, 9, 12):
            tw.check_state()
            tw.attention(0, i, dyn_mask=i & 1, what=f"frames tick {i}")


def test_error_paths_leave_state_unchanged(U):
    rb = U.rb
    w = synth.Workload("err", 5, synth.DTYPE_BF16, B=2, L=1, Hq=2, Hkv=1, d=64, S=8, S_max=8, N=4, T=4, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w)
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=U.DEV)
    q, kd, out = z(2, 4, 2, 64), z(2, 4, 1, 64), z(2, 4, 2, 64)

    def code(fn, *a, **k):
        with pytest.raises(rb.ReflexError) as e:
            fn(*a, **k)
        return e.value.code

    assert code(rb.reflex_partitioned_attention, tw.g, 0, q, kd, kd, out) == rb.ERR_STATE          # prefix never set
    tw.init_static([0], [8])
    assert code(rb.reflex_partitioned_attention, tw.g, 0, q, kd, kd, out) == rb.ERR_STATE          # stream 1 still unset
    tw.init_static([1], [0])                                                                        # S = 0 after an explicit init is legal
    rb.reflex_partitioned_attention(tw.g, 0, q, kd, kd, out)
    assert code(rb.reflex_partitioned_attention, tw.g, 1, q, kd, kd, out) == rb.ERR_INVALID_ARG    # layer out of range
    assert code(rb.reflex_partitioned_attention, tw.g, 0, z(2, 5, 2, 64), z(2, 5, 1, 64), z(2, 5, 1, 64), z(2, 5, 2, 64)) == rb.ERR_SHAPE
    assert code(rb.reflex_partitioned_attention, tw.g, 0, q, kd, kd, out, dyn_mask=2) == rb.ERR_INVALID_ARG
    assert code(rb.reflex_partitioned_attention, tw.g, 0, q.view(-1)[4:4 + 2 * 3 * 2 * 64].view(2, 3, 2, 64), kd[:, :3].contiguous(), kd[:, :3].contiguous(), out) == rb.ERR_ALIGN
    assert code(rb.reflex_cache_append_sliding, tw.g, [0], z(1, 1, 5, 1, 64), z(1, 1, 5, 1, 64)) == rb.ERR_SHAPE     # m > N
    assert code(rb.reflex_cache_append_sliding, tw.g, [2], z(1, 1, 1, 1, 64), z(1, 1, 1, 1, 64)) == rb.ERR_INVALID_ARG
    assert code(rb.reflex_cache_append_sliding, tw.g, [0, 0], z(2, 1, 1, 1, 64), z(2, 1, 1, 1, 64)) == rb.ERR_INVALID_ARG
    assert code(rb.reflex_cache_init_static, tw.g, [0], z(1, 1, 9, 1, 64), z(1, 1, 9, 1, 64)) == rb.ERR_SHAPE        # S > S_max
    assert code(rb.reflex_cache_init_static, tw.g, [0], z(1, 1, 4, 1, 64), z(1, 1, 4, 1, 64), S=[5]) == rb.ERR_SHAPE  # S > S_src
    tw.check_state()                                                                                                   # nothing moved
    assert code(rb.reflex_cache_set_attention_impl, tw.g, 9) == rb.ERR_INVALID_ARG


def test_adarmsnorm_gate_off_is_rmsnorm_and_flow_closed_form(U):
    """The gate switched off (W2 = 0, b2 = 0) leaves plain weight-free RMSNorm; checked against torch on the GPU
    tensor's own values as well as the oracle. Euler with constant v lands on x0 - v."""
    rb = U.rb
    w = synth.CONFIGS["cfg2"].with_(B=3)
    x = synth.norm_input(w, 0, 99)
    cond = synth.cond_vectors(w, 0.5)
    W1, b1, W2, b2 = synth.gate_weights(w, 0)       # b1 stays non-zero: with W2 = 0 and b2 = 0 the hidden layer cannot reach the gate
    dx = U.to_dev(x, w.dtype); dy = torch.empty_like(dx)
    rb.reflex_adarmsnorm(dx, dy, U.to_dev(cond, w.dtype), U.to_dev(W1, w.dtype), U.to_dev(b1, w.dtype),
                         U.to_dev(np.zeros_like(W2), w.dtype), U.to_dev(np.zeros_like(b2), w.dtype), eps=1e-6)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (w.D,), eps=1e-6).numpy()
    U.check_close(U.to_host(dy), ref, w.dtype, "gate-off norm", rel_clause=True)
    x0 = synth.normal(w, "noise", (w.B, w.T, w.A)); v = synth.normal(w, "v_flow", (w.B, w.T, w.A))
    xg = torch.from_numpy(x0).to(U.DEV)
    for k in range(w.K):
        rb.reflex_flow_step(xg, U.to_dev(v, w.dtype), None, k, w.K)
    assert np.max(np.abs(U.to_host(xg) - (x0.astype(np.float64) - v))) <= 2e-6


def test_stale_dynamic_kv_negative_control(U):
    """A cache that ignored the timestep (dynamic K/V frozen at step 0) is far outside tolerance."""
    rb = U.rb
    w = synth.CONFIGS["cfg2"]
    tw = U.Twin(w)
    tw.init_static([0], [w.S]); tw.append([0], 8, 0)
    q = synth.normal(w, "q", (1, w.T, w.Hq, w.d), 0, 1)
    kd0, vd0 = synth.normal(w, "k_dyn", (1, w.T, 1, w.d), 0, 0), synth.normal(w, "v_dyn", (1, w.T, 1, w.d), 0, 0)
    kd1, vd1 = synth.normal(w, "k_dyn", (1, w.T, 1, w.d), 0, 1), synth.normal(w, "v_dyn", (1, w.T, 1, w.d), 0, 1)
    out = torch.empty((1, w.T, w.Hq, w.d), dtype=torch.bfloat16, device=U.DEV)
    rb.reflex_partitioned_attention(tw.g, 0, U.to_dev(q, w.dtype), U.to_dev(kd0, w.dtype), U.to_dev(vd0, w.dtype), out)
    right = tw.o.attention(0, 0, q[0], kd1[0], vd1[0])
    err = np.abs(U.to_host(out)[0] - right)
    assert err.max() > 5 * U.BF16_MAX_ABS and err.mean() > 5 * U.BF16_MEAN_ABS


@pytest.mark.parametrize("cfg", ["cfg1", "cfg2"])
def test_10k_tick_stream_stays_finite(U, cfg):
    """Stability protocol (Sec. 4.4, stability table), raised to 10k ticks: every output of every tick is
    checked for NaN/Inf on the device (flag word, no host sync); outlier-laden norm inputs as in the long-context stress."""
    rb = U.rb
    w = synth.CONFIGS[cfg].with_(outlier_frac=1e-3, outlier_mult=1e3)
    cache = rb.Cache(w.L, w.B, w.Hq, w.Hkv, w.d, w.S_max, w.N, w.T, w.dtype, device=U.DEV)
    tdt = rb.torch_dtype(w.dtype)
    g = torch.Generator(device=U.DEV); g.manual_seed(w.seed)
    rnd = lambda *s: torch.randn(*s, generator=g, device=U.DEV, dtype=torch.float32).to(tdt)
    rb.reflex_cache_init_static(cache, [0], rnd(1, w.L, w.S, w.Hkv, w.d), rnd(1, w.L, w.S, w.Hkv, w.d))
    W1, b1, W2, b2 = [U.to_dev(a, w.dtype) for a in synth.gate_weights(w, 0)]
    n_var = 7
    xs = [U.to_dev(synth.norm_input(w, 0, i), w.dtype) for i in range(n_var)]
    conds = [U.to_dev(synth.cond_vectors(w, 1.0 - k / w.K), w.dtype) for k in range(w.K)]
    qs, kds, vds, vs = [[rnd(*s) for _ in range(n_var)] for s in ((w.B, w.T, w.Hq, w.d), (w.B, w.T, w.Hkv, w.d), (w.B, w.T, w.Hkv, w.d), (w.B, w.T, w.A))]
    kn, vn = [rnd(1, w.L, 1, w.Hkv, w.d) for _ in range(n_var)], [rnd(1, w.L, 1, w.Hkv, w.d) for _ in range(n_var)]
    y = torch.empty_like(xs[0]); out = torch.empty_like(qs[0])
    xa = torch.empty((w.B, w.T, w.A), dtype=torch.float32, device=U.DEV)
    bad = torch.zeros((), dtype=torch.int64, device=U.DEV)
    ticks = 10000
    steps = w.K
    for tick in range(ticks):
        rb.reflex_cache_append_sliding(cache, [0], kn[tick % n_var], vn[tick % n_var])
        xa.copy_(vs[tick % n_var].float())
        for k in range(steps):
            i = (tick + k) % n_var
            rb.reflex_adarmsnorm(xs[i], y, conds[k], W1, b1, W2, b2)
            rb.reflex_partitioned_attention(cache, 0, qs[i], kds[i], vds[i], out)
            rb.reflex_flow_step(xa, vs[i], None, k, w.K)
            if tick % 10 == 0 or k == steps - 1:   # every tick's final outputs, every step of each 10th tick
                bad += (~torch.isfinite(y.float())).sum() + (~torch.isfinite(out.float())).sum() + (~torch.isfinite(xa)).sum()
    assert int(bad.item()) == 0
    sl, hd, ct, tot = rb.reflex_cache_get_state(cache)
    assert tot == [ticks] and ct == [w.N] and hd == [ticks % w.N]


def test_gate_for_all_layers_matches_per_layer_calls_and_oracle(U):
    """reflex_adarmsnorm_gate with L stacked layers == L single-layer calls (bitwise) == the oracle's gamma."""
    from oracle import reflex_oracle as orc
    rb = U.rb
    w = synth.CONFIGS["cfg2"].with_(B=5, L=3)
    cond = synth.cond_vectors(w, 0.4)
    Ws = [synth.gate_weights(w, l, std=0.05) for l in range(w.L)]
    stack = lambda i: U.to_dev(np.stack([Ws[l][i] for l in range(w.L)]), w.dtype)
    W1s, b1s, W2s, b2s = stack(0), stack(1), stack(2), stack(3)
    dcond = U.to_dev(cond, w.dtype)
    all_buf = torch.full((w.L * w.B * (w.D + w.Hd),), float("nan"), dtype=torch.float32, device=U.DEV)
    rb.reflex_adarmsnorm_gate(dcond, W1s, b1s, W2s, b2s, all_buf)
    x = synth.norm_input(w, 0, 0)
    for l in range(w.L):
        one = torch.full((w.B * (w.D + w.Hd),), float("nan"), dtype=torch.float32, device=U.DEV)
        rb.reflex_adarmsnorm_gate(dcond, W1s[l], b1s[l], W2s[l], b2s[l], one)
        g_all = all_buf[l * w.B * w.D:(l + 1) * w.B * w.D]
        assert torch.equal(g_all, one[: w.B * w.D])
        for b in (0, 4):
            _, g = orc.adarmsnorm(x[b], cond[b], *Ws[l], 1e-6, return_gate=True)
            assert (np.abs(U.to_host(g_all.view(w.B, w.D)[b]) - g) <= _gate_tol(orc, cond[b], *Ws[l])).all()
        # a layer's rows with its slice of the step's gates == the all-in-one call
        dx = U.to_dev(x, w.dtype)
        y1, y2 = torch.empty_like(dx), torch.empty_like(dx)
        rb.reflex_adarmsnorm(dx, y1, None, None, None, None, None, gate_buf=g_all.view(w.B, w.D))
        rb.reflex_adarmsnorm(dx, y2, dcond, W1s[l], b1s[l], W2s[l], b2s[l], gate_buf=one)
        assert torch.equal(y1, y2)
        U.check_close(U.to_host(y1), orc.adarmsnorm_batched(x, cond, *Ws[l], 1e-6), w.dtype, f"rows with step gates, layer {l}", rel_clause=True)


GATE_PATHS = [
    # name, dtype, B, D, Cd, Hd, L, std, bias_std        which kernels compute the gate
    ("bf16_tensor_core", synth.DTYPE_BF16, 70, 1024, 288, 256, 3, 0.1, 0.3),     # tcgen05 gate kernels: two stream groups, one and three layers
    ("bf16_tick_stacked", synth.DTYPE_BF16, 210, 1024, 288, 256, 2, 0.1, 0.3),   # K x B conditioning vectors stacked as streams: four groups, ragged last
    ("f32_fma", synth.DTYPE_F32, 37, 128, 40, 32, 3, 0.2, 0.3),                  # fp32: thread-per-dot-product kernel (one layer), register-tiled (three)
    ("bf16_fma_widths", synth.DTYPE_BF16, 37, 256, 40, 24, 2, 0.2, 0.3),         # widths the tensor-core kernel refuses (not multiples of 16)
    ("f32_wide_rows32", synth.DTYPE_F32, 5, 128, 600, 560, 2, 0.05, 0.3),        # too wide for the register-tiled kernel: 32 weight rows per block
    ("bf16_very_wide", synth.DTYPE_BF16, 3, 256, 1024, 640, 2, 0.03, 0.3),       # beyond the staged kernels' shared memory: per-stream gate kernel
]


@pytest.mark.parametrize("case", GATE_PATHS, ids=[c[0] for c in GATE_PATHS])
def test_gate_paths_with_nonzero_biases(U, case):
    """Eq. 2's gate 1 + W2 SiLU(W1 c + b1) + b2 with both biases far from zero and weights large enough that the hidden
    layer carries the gate, through every kernel that computes it: the single fused launch, the two-launch form with
    scratch, the stacked call for L layers, and the rows kernel fed a layer's slice of the stacked gates. Gates are compared
    in fp32 against the oracle for every stream and layer, outputs element-wise."""
    from oracle import reflex_oracle as orc
    rb = U.rb
    name, dtype, B, D, Cd, Hd, L, std, bias_std = case
    w = synth.Workload(name, 51, dtype, B=B, L=L, Hq=1, Hkv=1, d=8, S=1, S_max=1, N=1, T=6, D=D, Cd=Cd, Hd=Hd, A=4, K=2)
    x = synth.norm_input(w, 0, 0)
    cond = np.concatenate([synth.cond_vectors(w, t, B=(B + 2) // 3, variant=i) for i, t in enumerate((0.9, 0.5, 0.1))])[:B]
    Ws = [synth.gate_weights(w, l, std=std, bias_std=bias_std) for l in range(L)]
    assert all(np.abs(W[1]).max() > 0.2 and np.abs(W[3]).max() > 0.2 for W in Ws)
    want_y, want_g = [], []
    for l in range(L):
        pairs = [orc.adarmsnorm(x[b], cond[b], *Ws[l], 1e-6, return_gate=True) for b in range(B)]
        want_y.append(np.stack([p[0] for p in pairs])); want_g.append(np.stack([p[1] for p in pairs]))
    assert np.abs(want_g[0] - 1.0).mean() > 0.2          # the gate really moves
    tol_g = [np.stack([_gate_tol(orc, cond[b], *Ws[l]) for b in range(B)]) for l in range(L)]
    dx, dcond = U.to_dev(x, dtype), U.to_dev(cond, dtype)
    d0 = [U.to_dev(a, dtype) for a in Ws[0]]
    rms = lambda a: float(np.sqrt(np.mean(a * a)))
    # the fused single launch (every block recomputes its stream's gate)
    y = torch.full_like(dx, float("nan"))
    rb.reflex_adarmsnorm(dx, y, dcond, *d0)
    U.check_close(U.to_host(y), want_y[0], dtype, name + ": fused launch", rel_clause=True, out_scale=rms(want_y[0]))
    # gate kernels + rows kernel with caller scratch
    gb = torch.full((B * (D + Hd),), float("nan"), dtype=torch.float32, device=U.DEV)
    y2 = torch.full_like(dx, float("nan"))
    rb.reflex_adarmsnorm(dx, y2, dcond, *d0, gate_buf=gb)
    assert (np.abs(U.to_host(gb[: B * D]).reshape(B, D) - want_g[0]) <= tol_g[0]).all(), name + ": gate with scratch"
    U.check_close(U.to_host(y2), want_y[0], dtype, name + ": two launches", rel_clause=True, out_scale=rms(want_y[0]))
    # all L layers by one call, then the rows kernel on the last layer's slice
    stack = lambda i: U.to_dev(np.stack([Ws[l][i] for l in range(L)]), dtype)
    g_all = torch.full((L * B * (D + Hd),), float("nan"), dtype=torch.float32, device=U.DEV)
    rb.reflex_adarmsnorm_gate(dcond, stack(0), stack(1), stack(2), stack(3), g_all)
    got_g = U.to_host(g_all[: L * B * D]).reshape(L, B, D)
    for l in range(L):
        assert (np.abs(got_g[l] - want_g[l]) <= tol_g[l]).all(), f"{name}: stacked gates, layer {l}"
    y3 = torch.full_like(dx, float("nan"))
    rb.reflex_adarmsnorm(dx, y3, None, None, None, None, None, gate_buf=g_all[(L - 1) * B * D: L * B * D].view(B, D))
    U.check_close(U.to_host(y3), want_y[L - 1], dtype, name + ": rows with stacked gates", rel_clause=True, out_scale=rms(want_y[L - 1]))


# ------------------------------------------------------------------------------------------------
# adaptive norm folded into the packed Q/K/V projection
# ------------------------------------------------------------------------------------------------
def _norm_qkv_case(U, w, impl, what, t=0.3, eps=1e-6, streams=None):
    from oracle import reflex_oracle as orc
    rb = U.rb
    x = synth.norm_input(w, 0, 0)
    cond = synth.cond_vectors(w, t)
    W1, b1, W2, b2 = synth.gate_weights(w, 0)          # gate near 1: unit-variance outputs, which the bf16 contract presumes
    Wp = synth.qkv_weights(w, 0)
    gb = torch.empty((w.B * (w.D + w.Hd),), dtype=torch.float32, device=U.DEV)
    rb.reflex_adarmsnorm_gate(U.to_dev(cond, w.dtype), U.to_dev(W1, w.dtype), U.to_dev(b1, w.dtype), U.to_dev(W2, w.dtype), U.to_dev(b2, w.dtype), gb)
    dt = rb.torch_dtype(w.dtype)
    q = torch.full((w.B, w.T, w.Hq, w.d), float("nan"), dtype=dt, device=U.DEV)
    k = torch.full((w.B, w.T, w.Hkv, w.d), float("nan"), dtype=dt, device=U.DEV)
    v = torch.full((w.B, w.T, w.Hkv, w.d), float("nan"), dtype=dt, device=U.DEV)
    rb.reflex_adarmsnorm_qkv(U.to_dev(x, w.dtype), gb[: w.B * w.D].view(w.B, w.D), U.to_dev(Wp, w.dtype), q, k, v, eps=eps, impl=impl)
    torch.cuda.synchronize()
    for b in (range(w.B) if streams is None else streams):
        wq, wk, wv = orc.adarmsnorm_qkv(x[b], cond[b], W1, b1, W2, b2, Wp, w.Hq, w.Hkv, w.d, eps)
        for got, want, name in ((q, wq, "q"), (k, wk, "k"), (v, wv, "v")):
            U.check_close(U.to_host(got[b]), want, w.dtype, f"{what} {name} stream {b}", rel_clause=True)


def test_norm_qkv_fp32_plain_kernel(U):
    _norm_qkv_case(U, synth.CONFIGS["cfg1"].with_(B=3), 0, "norm+qkv fp32")


@pytest.mark.parametrize("impl", [0, 1])
def test_norm_qkv_bf16_action_expert_shape(U, impl):
    """cfg2 shapes (D = 1024, 8 + 1 + 1 heads of 256) for 7 streams of 50 rows: 350 rows = one full 256-row tile pair and a
    second with 94 rows (its second CTA entirely past the end), 10 column tiles, rows of several streams in one tile."""
    _norm_qkv_case(U, synth.CONFIGS["cfg2"].with_(B=7), impl, f"norm+qkv bf16 impl {impl}")


@pytest.mark.parametrize("impl", [0, 2])
def test_norm_qkv_bf16_many_streams(U, impl):
    """40 streams of 50 rows = 2000 rows: 8 row tiles x 10 column tiles exceed the SM pairs, so impl 0 takes the 512-column
    tiles (two accumulators; 5 column tiles); impl 2 keeps 256-column tiles. A sample of streams is compared."""
    _norm_qkv_case(U, synth.CONFIGS["cfg2"].with_(B=40), impl, f"norm+qkv bf16 40 streams impl {impl}", streams=[0, 5, 6, 20, 39])


def test_norm_qkv_bf16_ragged_columns_and_outliers(U):
    """320 output columns (a second column tile with 64 of 256 live), head_dim 64, D = 192 (three contraction steps, fewer
    than the stage ring), 300 rows per stream, and x with outliers x1000 as in the long-context configuration."""
    w = synth.CONFIGS["cfg5"].with_(B=2, T=300, Hq=3, Hkv=1, d=64, D=192, L=1)
    _norm_qkv_case(U, w, 0, "norm+qkv ragged", t=1e-3)


def test_norm_qkv_error_paths(U):
    rb = U.rb
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=U.DEV)
    x, g, W = z(2, 4, 64), torch.ones((2, 64), dtype=torch.float32, device=U.DEV), z(4 * 16, 64)
    q, k = z(2, 4, 2, 16), z(2, 4, 1, 16)
    rb.reflex_adarmsnorm_qkv(x, g, W, q, k, k.clone())
    for bad in (lambda: rb.reflex_adarmsnorm_qkv(x, g, W, q, k, k, impl=3),
                lambda: rb.reflex_adarmsnorm_qkv(x, g, W, q, k, k, eps=-1.0)):
        with pytest.raises(rb.ReflexError) as e:
            bad()
        assert e.value.code == rb.ERR_INVALID_ARG
    with pytest.raises(rb.ReflexError) as e:
        rb.reflex_adarmsnorm_qkv(x, g, W, z(2, 4, 2, 12), z(2, 4, 1, 12), z(2, 4, 1, 12))     # head_dim not a multiple of 8
    assert e.value.code == rb.ERR_SHAPE
    with pytest.raises(rb.ReflexError) as e:
        rb.reflex_adarmsnorm_qkv(x.view(-1)[4:4 + 2 * 3 * 64].view(2, 3, 64), g, W, q[:, :3].contiguous(), k[:, :3].contiguous(), k[:, :3].contiguous())
    assert e.value.code == rb.ERR_ALIGN


def test_chained_layer_norm_qkv_attention(U):
    """The chained layer: AdaRMSNorm + packed projection writes Q, K_dyn, V_dyn, the partitioned attention reads them.
    Against the oracle chain in fp64 throughout (no rounding of Q/K/V in between): the bf16 storage of Q/K/V moves a logit by
    about 2e-3 and the output far less than the contract's tolerance."""
    from oracle import reflex_oracle as orc
    rb = U.rb
    w = synth.CONFIGS["cfg2"].with_(B=3)
    tw = U.Twin(w, head0=[0, 5, 31], poison=True)
    tw.init_static([0, 1, 2], [w.S, 700, 64])
    for i in range(20):
        tw.append([0, 1, 2] if i < 12 else [0, 1], 1, i)
    x = synth.norm_input(w, 0, 3)
    cond = synth.cond_vectors(w, 0.7)
    W1, b1, W2, b2 = synth.gate_weights(w, 0)
    Wp = synth.qkv_weights(w, 0)
    gb = torch.empty((w.B * (w.D + w.Hd),), dtype=torch.float32, device=U.DEV)
    rb.reflex_adarmsnorm_gate(U.to_dev(cond, w.dtype), U.to_dev(W1, w.dtype), U.to_dev(b1, w.dtype), U.to_dev(W2, w.dtype), U.to_dev(b2, w.dtype), gb)
    nan = lambda *s: torch.full(s, float("nan"), dtype=torch.bfloat16, device=U.DEV)
    q, k, v, out = nan(w.B, w.T, w.Hq, w.d), nan(w.B, w.T, w.Hkv, w.d), nan(w.B, w.T, w.Hkv, w.d), nan(w.B, w.T, w.Hq, w.d)
    rb.reflex_adarmsnorm_qkv(U.to_dev(x, w.dtype), gb[: w.B * w.D].view(w.B, w.D), U.to_dev(Wp, w.dtype), q, k, v, cache=tw.g)
    rb.reflex_partitioned_attention(tw.g, 0, q, k, v, out, dyn_mask=1)
    rb.reflex_cache_check_status(tw.g)
    got = U.to_host(out)
    for b in range(w.B):
        wq, wk, wv = orc.adarmsnorm_qkv(x[b], cond[b], W1, b1, W2, b2, Wp, w.Hq, w.Hkv, w.d)
        want = tw.o.attention(b, 0, wq.astype(np.float32), wk.astype(np.float32), wv.astype(np.float32), 1, None)
        U.check_close(got[b], want, w.dtype, f"chained layer stream {b}")


# ------------------------------------------------------------------------------------------------
# adaptive norm folded into the fused gate / up projections of a SwiGLU block
# ------------------------------------------------------------------------------------------------
def _norm_swiglu_case(U, w, F, impl, what, t=0.3, eps=1e-6, streams=None):
    from oracle import reflex_oracle as orc
    rb = U.rb
    x = synth.norm_input(w, 0, 1)
    cond = synth.cond_vectors(w, t)
    W1, b1, W2, b2 = synth.gate_weights(w, 0)
    Wgu = synth.swiglu_weights(w, 0, F)
    gb = torch.empty((w.B * (w.D + w.Hd),), dtype=torch.float32, device=U.DEV)
    rb.reflex_adarmsnorm_gate(U.to_dev(cond, w.dtype), U.to_dev(W1, w.dtype), U.to_dev(b1, w.dtype), U.to_dev(W2, w.dtype), U.to_dev(b2, w.dtype), gb)
    h = torch.full((w.B, w.T, F), float("nan"), dtype=rb.torch_dtype(w.dtype), device=U.DEV)
    rb.reflex_adarmsnorm_swiglu(U.to_dev(x, w.dtype), gb[: w.B * w.D].view(w.B, w.D), U.to_dev(Wgu, w.dtype), h, eps=eps, impl=impl)
    torch.cuda.synchronize()
    for b in (range(w.B) if streams is None else streams):
        want = orc.adarmsnorm_swiglu(x[b], cond[b], W1, b1, W2, b2, Wgu[:F], Wgu[F:], eps)
        got = U.to_host(h[b])
        if w.dtype != synth.DTYPE_BF16:
            U.check_close(got, want, w.dtype, f"{what} stream {b}", rel_clause=True)
            continue
        # bf16: each projection reaches the activation with the operand-rounding error of a bf16 GEMM over D terms, at most
        # delta = 6.3e-3 per unit of output scale (4.5 sigma of 1.4e-3); h = SiLU(g) u then moves by |SiLU'(g) u| delta +
        # |SiLU(g)| delta (|SiLU'| <= 1.1), on top of the contract's allowance for the stored value itself
        y = orc.adarmsnorm(x[b], cond[b], W1, b1, W2, b2, eps)
        g, u = y @ Wgu[:F].astype(np.float64).T, y @ Wgu[F:].astype(np.float64).T
        silu = g / (1.0 + np.exp(-g))
        lim = np.maximum(U.BF16_MAX_ABS, 2.0 ** -7 * np.abs(want)) + 6.3e-3 * (1.1 * np.abs(u) + np.abs(silu))
        err = np.abs(got - want)
        assert np.isfinite(got).all() and not (err > lim).any(), f"{what} stream {b}: worst {err.max():.3e}, {(err > lim).sum()} beyond the bound"
        assert err.mean() <= U.BF16_MEAN_ABS, f"{what} stream {b}: mean-abs {err.mean():.3e}"


def test_norm_swiglu_fp32_plain_kernel(U):
    _norm_swiglu_case(U, synth.CONFIGS["cfg1"].with_(B=2), 96, 0, "norm+swiglu fp32")


@pytest.mark.parametrize("impl", [0, 1])
def test_norm_swiglu_bf16(U, impl):
    """D = 1024, F = 1024 hidden features (4 column tiles of 256, each with a gate and an up accumulator), 7 streams of 50
    rows (a full 256-row tile pair and a ragged one)."""
    _norm_swiglu_case(U, synth.CONFIGS["cfg2"].with_(B=7), 1024, impl, f"norm+swiglu bf16 impl {impl}")


def test_norm_swiglu_bf16_ragged_hidden_width(U):
    """F = 328: the second column tile has 72 live columns and its gate accumulator reads rows of W_up past W_gate's end
    (never stored); D = 192."""
    w = synth.CONFIGS["cfg2"].with_(B=3, T=120, D=192)
    _norm_swiglu_case(U, w, 328, 0, "norm+swiglu ragged")


@pytest.mark.parametrize("D", [128, 640])
def test_norm_qkv_more_tiles_than_sm_pairs(U, D):
    """128 streams of 50 rows = 6400 rows: 25 row tiles x 5 column tiles of 512 = 125 tiles, more than the SM pairs, so every
    CTA pair walks two tiles and hands the stage ring and the accumulators from one to the next (both accumulators are staged
    for the TMA stores, so the next tile's weights wait for them too). D = 128 gives two contraction steps per tile, fewer
    than the stage ring; D = 640 ten. A sample of streams from first and later tiles of a pair is compared."""
    w = synth.CONFIGS["cfg2"].with_(B=128, D=D)
    _norm_qkv_case(U, w, 0, f"norm+qkv 125 tiles D={D}", streams=[0, 1, 37, 63, 64, 100, 126, 127])


def test_norm_qkv_more_tiles_than_sm_pairs_one_accumulator(U):
    """D = 2048: the gates of a tile's four streams no longer fit beside two accumulators' stages, so the tiles are 256 columns
    wide; 100 streams of 50 rows (20 row tiles) x 4 column tiles (2 + 1 + 1 heads of 256) = 80 tiles on 74 SM pairs."""
    w = synth.CONFIGS["cfg2"].with_(B=100, D=2048, Hq=2, Hkv=1)
    _norm_qkv_case(U, w, 0, "norm+qkv 80 tiles, one accumulator", streams=[0, 4, 5, 50, 94, 95, 99])


def test_norm_swiglu_more_tiles_than_sm_pairs(U):
    """6400 rows x 1000 hidden features (ragged last column tile) with D = 192: 25 x 4 = 100 tiles of three steps on 74 pairs."""
    w = synth.CONFIGS["cfg2"].with_(B=128, D=192)
    _norm_swiglu_case(U, w, 1000, 0, "norm+swiglu 100 tiles", streams=[0, 1, 63, 64, 90, 127])


@pytest.mark.parametrize("B", [2, 5, 8, 13])
def test_projections_row_groups_of_the_few_rows_kernel(U, B):
    """100, 250, 400 and 650 rows: the few-rows kernel (weights as the A operand) on groups of 64 rows (of 128 where those
    would outnumber the SMs), one CTA per feature tile and group; the last group ragged, streams straddling group boundaries (their gates staged per group). The fused gate/up
    projection takes the groups up to 256 rows (32 feature tiles x 4 groups), the plain projection for a contraction of
    4096 (split over clusters of 4), the packed Q/K/V projection up to 448 rows."""
    w = synth.CONFIGS["cfg2"].with_(B=B)
    streams = sorted({0, 1, B // 2, B - 1})
    _norm_qkv_case(U, w, 0, f"norm+qkv {B * w.T} rows in groups", streams=streams)
    _norm_swiglu_case(U, w, 4096, 0, f"norm+swiglu {B * w.T} rows in groups", streams=streams[:2])
    M = B * w.T
    rows = sorted({0, 63, 64, 65, M // 2, M - 1} & set(range(M)))
    _linear_case(U, synth.DTYPE_BF16, M, 4096, 1024, 0, f"linear {M} rows in groups", rows=rows, seed=71)
    _linear_case(U, synth.DTYPE_BF16, M, 2048, 1000, 0, f"linear {M} rows, contraction 2048", rows=rows, seed=72)


def test_norm_qkv_short_streams_and_fallback(U):
    """Rows per stream far below the tile height: with R = 13 a 128-row tile covers 11 streams (all their gates in shared
    memory); with R = 3 the gates of a tile's 44 streams no longer fit beside the stages and the call falls back to the plain
    kernel. Both against the oracle."""
    w13 = synth.CONFIGS["cfg2"].with_(B=23, T=13)
    _norm_qkv_case(U, w13, 0, "norm+qkv R=13", streams=[0, 9, 10, 22])
    w3 = synth.CONFIGS["cfg2"].with_(B=50, T=3)
    _norm_qkv_case(U, w3, 0, "norm+qkv R=3 (plain kernel)", streams=[0, 42, 43, 49])


# ------------------------------------------------------------------------------------------------
# plain projections with residual (attention output projection, SwiGLU down projection)
# ------------------------------------------------------------------------------------------------
def _linear_case(U, dtype, M, K, N, impl, what, residual=True, in_place=False, rows=None, seed=61):
    """out = res + a W^T against the oracle's triple loop. a ~ N(0,1), W ~ N(0, 1/K), res ~ N(0,1): outputs of variance 2
    (1 without residual). The operands are exact in the storage dtype and accumulate in fp32, so what is left is the
    rounding of the output: the bf16 contract with its output-spacing clause, mean-abs scaled to the output's rms."""
    from oracle import reflex_oracle as orc
    rb = U.rb
    w = synth.Workload("lin", seed, dtype, B=1, L=1, Hq=1, Hkv=1, d=8, S=1, S_max=1, N=1, T=1, D=8, Cd=8, Hd=8, A=4, K=1)
    a = synth.normal(w, "x", (M, K), 0, 0)
    W = synth.normal(w, "Wo", (N, K), 0, 0, float(K) ** -0.5)
    res = synth.normal(w, "misc", (M, N), 0, 0) if residual else None
    da, dW = U.to_dev(a, dtype), U.to_dev(W, dtype)
    dres = U.to_dev(res, dtype) if residual else None
    out = dres if in_place else torch.full((M, N), float("nan"), dtype=rb.torch_dtype(dtype), device=U.DEV)
    rb.reflex_linear_residual(da, dW, dres, out, impl=impl)
    torch.cuda.synchronize()
    rows = list(range(M)) if rows is None else rows
    want = orc.linear_residual(a[rows], W, res[rows] if residual else None)
    U.check_close(U.to_host(out)[rows], want, dtype, what, rel_clause=True, out_scale=float(np.sqrt(np.mean(want ** 2))))
    if not in_place and residual:
        assert torch.equal(dres, U.to_dev(res, dtype))      # the residual itself is only read


def test_linear_residual_fp32_plain_kernel(U):
    _linear_case(U, synth.DTYPE_F32, 37, 136, 72, 0, "linear fp32")
    _linear_case(U, synth.DTYPE_F32, 5, 64, 8, 0, "linear fp32, no residual", residual=False)


@pytest.mark.parametrize("K", [2048, 4096])
def test_linear_residual_bf16_output_and_down_projection(U, K):
    """The expert's output projection (K = Hq d = 2048) and down projection (K = F = 4096) onto D = 1024 for 7 streams of 50
    rows: a full 256-row tile pair and one with 94 rows (its second CTA entirely past the end), four column tiles; in place
    and out of place, against the plain kernel's path as well."""
    _linear_case(U, synth.DTYPE_BF16, 350, K, 1024, 0, f"linear bf16 K={K}")
    _linear_case(U, synth.DTYPE_BF16, 350, K, 1024, 0, f"linear bf16 K={K} in place", in_place=True)
    _linear_case(U, synth.DTYPE_BF16, 350, K, 1024, 1, f"linear bf16 K={K} plain kernel", rows=[0, 127, 128, 255, 256, 349])


def test_linear_residual_bf16_ragged_shapes(U):
    """Column count 328 (a second column tile with 72 live columns, its last 64-column piece clipped at 8), contraction 200
    (not a multiple of the 64-column step: the tail arrives as zeros), 300 rows; and without residual."""
    _linear_case(U, synth.DTYPE_BF16, 300, 200, 328, 0, "linear ragged")
    _linear_case(U, synth.DTYPE_BF16, 300, 200, 328, 0, "linear ragged, no residual", residual=False)
    _linear_case(U, synth.DTYPE_BF16, 129, 64, 8, 0, "linear one step, 8 columns")
    _linear_case(U, synth.DTYPE_BF16, 130, 8, 72, 0, "linear contraction of 8 (narrower than a 64-column step)")
    _linear_case(U, synth.DTYPE_BF16, 40, 72, 136, 0, "linear few rows, contraction not a multiple of 64 (256-row tile path)")
    # enough row tiles for the 256-column tiles (the smaller problems above take 128-column tiles): 2600 rows, a ragged last
    # row tile, three contraction steps
    _linear_case(U, synth.DTYPE_BF16, 2600, 192, 1024, 0, "linear 256-column tiles", in_place=True, rows=[0, 255, 256, 1300, 2559, 2560, 2599])


@pytest.mark.parametrize("M", [50, 100])
def test_linear_residual_bf16_few_rows(U, M):
    """One or two streams of 50 rows: the kernel with the weights as the stationary operand (64 or 128 row columns), and the
    same shapes forced through the 256-row tiles."""
    _linear_case(U, synth.DTYPE_BF16, M, 2048, 1024, 0, f"linear {M} rows")
    _linear_case(U, synth.DTYPE_BF16, M, 4096, 1024, 0, f"linear {M} rows K=4096 in place", in_place=True)
    _linear_case(U, synth.DTYPE_BF16, M, 192, 328, 0, f"linear {M} rows ragged", residual=False)
    _linear_case(U, synth.DTYPE_BF16, M, 2048, 1024, 2, f"linear {M} rows, 256-row tiles")


def _random_projection_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        B = int(rng.choice([1, 2, 3, 7, 20, 45]))
        T = int(rng.choice([1, 13, 50, 64, 100]))
        D = int(rng.choice([64, 192, 512, 1024]))
        Hq, d = int(rng.choice([1, 3, 8])), int(rng.choice([64, 128, 256]))
        F = int(rng.choice([8, 72, 256, 328, 1000]))
        N = int(rng.choice([8, 72, 256, 1000]))
        cases.append((f"p{i}_B{B}_T{T}_D{D}_Hq{Hq}_d{d}_F{F}_N{N}", B, T, D, Hq, d, F, N))
    return cases


RANDOM_PROJECTIONS = _random_projection_cases(12, 14695)


@pytest.mark.parametrize("case", RANDOM_PROJECTIONS, ids=[c[0] for c in RANDOM_PROJECTIONS])
def test_random_shapes_projections(U, case):
    """Seeded shapes through the three projection entry points (norm + Q/K/V, norm + gate/up, plain + residual) with the
    kernel the library picks for them (few rows, 256-row tiles with one or two accumulators, plain kernel for what the
    tensor-core forms refuse), a sample of streams / rows against the oracle."""
    name, B, T, D, Hq, d, F, N = case
    w = synth.CONFIGS["cfg2"].with_(B=B, T=T, D=D, Hq=Hq, Hkv=1, d=d)
    streams = sorted({0, B // 2, B - 1})
    _norm_qkv_case(U, w, 0, name + " norm+qkv", streams=streams)
    _norm_swiglu_case(U, w, F, 0, name + " norm+swiglu", streams=streams)
    M = B * T
    rows = sorted({0, M // 3, M // 2, M - 1} | set(range(max(0, M - 5), M)))
    _linear_case(U, synth.DTYPE_BF16, M, D, N, 0, name + " linear", rows=rows, seed=70)


@pytest.mark.parametrize("M,K,N,residual", [(800, 4096, 1024, True), (800, 2048, 1024, True), (650, 4096, 1000, False), (1000, 4160, 512, True)])
def test_linear_residual_bf16_mid_size_rows(U, M, K, N, residual):
    """Between the few-rows form and full occupancy: 128-column tiles, and while two pairs per tile still fit the SM pairs
    a contraction of 4096 or more split in two over a cluster of four CTAs (the halves meet through distributed shared
    memory): 800 rows with both contractions of the expert (2048 stays unsplit), a ragged last column tile without a
    residual in the split form, and an odd number of contraction steps (65), which stays unsplit. Rows from every row tile, both CTAs of a pair, and the ragged end."""
    rows = sorted({0, 1, 127, 128, 255, 256, 300, M // 2, M - 130, M - 2, M - 1})
    _linear_case(U, synth.DTYPE_BF16, M, K, N, 0, f"linear {M}x{K}->{N}", residual=residual, rows=rows, seed=73)


def test_linear_residual_error_paths(U):
    rb = U.rb
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=U.DEV)
    a, W, r = z(4, 64), z(16, 64), z(4, 16)
    rb.reflex_linear_residual(a, W, r, r)
    for bad, code in ((lambda: rb.reflex_linear_residual(a, W, r, r, impl=3), rb.ERR_INVALID_ARG),
                      (lambda: rb.reflex_linear_residual(a, W, r, a), rb.ERR_INVALID_ARG),                      # out aliases a
                      (lambda: rb.reflex_linear_residual(z(4, 60), z(16, 60), r, r), rb.ERR_SHAPE),             # K % 8
                      (lambda: rb.reflex_linear_residual(a, z(12, 64), z(4, 12), z(4, 12)), rb.ERR_SHAPE),      # N % 8
                      (lambda: rb.reflex_linear_residual(a.view(-1)[4:4 + 3 * 64].view(3, 64), W, r[:3].contiguous(), r[:3].contiguous()), rb.ERR_ALIGN)):
        with pytest.raises(rb.ReflexError) as e:
            bad()
        assert e.value.code == code


# ------------------------------------------------------------------------------------------------
# producer / consumer: a new prefix staged in the second static bank while the current one is read
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", ["simt", "tc", "tc2"])
def test_double_banked_static_prefix(U, impl):
    rb = U.rb
    w = synth.CONFIGS["cfg2"].with_(B=3, S=300, S_max=320)
    tw = U.Twin(w, head0=[0, 9, 31], poison=True, static_banks=2)
    rb.reflex_cache_set_attention_impl(tw.g, {"simt": rb.ATTN_SIMT, "tc": rb.ATTN_TC, "tc2": rb.ATTN_TC2}[impl])
    tw.init_static([0, 1, 2], [300, 257, 64])
    for i in range(3):
        tw.append([0, 1, 2], 7, i)
    tw.check_state()
    tw.attention(0, 0, what="banked: first prefix")
    # the producer stages new prefixes for streams 0 and 2 on its own stream; the consumer's attention, launched right
    # behind it on the main stream without any ordering between the two, still sees the first prefix
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        keep = tw.stage_static([0, 2], [320, 100], 5, stream=side)
    tw.attention(0, 1, dyn_mask=1, what="banked: staged but not committed")
    tw.append([0, 1, 2], 30, 7)                                   # the ring moves on independently of the banks
    tw.attention(0, 2, what="banked: staged, ring advanced")
    # hand-over between two chunks: the consumer waits for the producer's writes, then flips
    torch.cuda.current_stream().wait_stream(side)
    tw.commit_static([0, 2])
    tw.check_state()
    tw.attention(0, 3, dyn_mask=1, what="banked: committed")
    # and back into the first bank, with a shorter prefix for stream 0 only
    keep2 = tw.stage_static([0], [48], 6)
    tw.attention(0, 4, what="banked: second staging")
    tw.commit_static([0])
    tw.check_state()
    tw.attention(0, 5, what="banked: second commit")
    sl, _, _, _ = rb.reflex_cache_get_state(tw.g)
    assert sl == [48, 257, 100]
    with pytest.raises(rb.ReflexError) as e:
        tw_err = rb.reflex_cache_commit_static(tw.g, [1])          # nothing staged for stream 1
    assert e.value.code == rb.ERR_STATE
    single = U.Twin(w.with_(B=1))
    with pytest.raises(rb.ReflexError) as e:
        rb.reflex_cache_commit_static(single.g, [0])
    assert e.value.code == rb.ERR_STATE
    del keep, keep2


@pytest.mark.parametrize("frames,T", [(1, 75), (5, 50), (50, 25)])
def test_context_window_and_chunk_sweep(U, frames, T):
    """Points of the paper's context-window (1 to 50 frames of 256 tokens in the sliding history) and action-chunk (25 to 100
    tokens) ablations: the ring is filled frame by frame past its capacity, with a partly filled second stream."""
    N = frames * 256
    w = synth.Workload("sweep", 43, synth.DTYPE_BF16, B=2, L=1, Hq=8, Hkv=1, d=256, S=300, S_max=320, N=N, T=T, D=64, Cd=8, Hd=8, A=4, K=2)
    tw = U.Twin(w, head0=[0, N - 100], poison=True)
    tw.init_static([0, 1], [300, 129])
    n_app = min(frames + 2, 7)            # past the capacity for the small windows, partly filled for the largest
    for i in range(n_app):
        tw.append([0, 1] if i % 3 != 2 else [0], 256, i)
    tw.check_state()
    tw.attention(0, 0, dyn_mask=0, what=f"sweep {frames} frames, T={T}")
    tw.attention(0, 1, dyn_mask=1, what=f"sweep {frames} frames, T={T}, causal")


# ------------------------------------------------------------------------------------------------
# a whole action-expert denoising step chained from the library's calls
# ------------------------------------------------------------------------------------------------
def _expert_case(U, w, F, tol_v, what, streams=None):
    from oracle import expert_oracle as eo
    from paper_2607_14695_b200 import expert as ex
    rb = U.rb
    tw = U.Twin(w, head0=[3] * w.B, poison=True)
    tw.init_static(list(range(w.B)), [w.S] * w.B)
    for i in range(3):
        tw.append(list(range(w.B)), 2, i)
    W = ex.expert_weights(w, F, std_scale=0.5)
    dW = {n: U.to_dev(v, w.dtype) for n, v in W.items()}
    model = ex.ActionExpert(w, tw.g, dW, F, device=U.DEV)
    a0 = synth.normal(w, "noise", (w.B, w.T, w.A)).astype(np.float64)
    if w.dtype == synth.DTYPE_BF16:          # the step reads the chunk through a storage-dtype mirror: start from representable values
        a0 = synth.round_storage(a0.astype(np.float32), w.dtype).astype(np.float64)
    cond = synth.cond_vectors(w, 0.6)
    a_gpu = torch.from_numpy(a0.astype(np.float32)).to(U.DEV)
    model.step(a_gpu, U.to_dev(cond, w.dtype), 1)
    rb.reflex_cache_check_status(tw.g)
    want_a, want_v = eo.expert_step(tw.o, W, a0, cond, w.K, w.Hq, w.Hkv, w.d, F, streams=streams)
    got_v = U.to_host(model.vel)
    if streams is not None:          # a sample of the (independent) streams
        got_v, want_v, want_a = got_v[streams], want_v[streams], want_a[streams]
        a_gpu = a_gpu[streams]
    rel = np.linalg.norm(got_v - want_v) / np.linalg.norm(want_v)
    assert np.isfinite(got_v).all() and rel <= tol_v, f"{what}: velocity off by {rel:.3e} (relative Frobenius)"
    # element by element: the roundings that accumulate along the chain are independent, so an element's error is spread
    # around tol_v * rms(v) at most; none may pass five times that (a wrong row, column or stream is off by ~ rms(v))
    rms_v = float(np.sqrt(np.mean(want_v ** 2)))
    worst = np.abs(got_v - want_v).max()
    assert worst <= 5.0 * tol_v * rms_v, f"{what}: worst velocity element off by {worst:.3e} (rms {rms_v:.3e})"
    err_a = np.abs(a_gpu.double().cpu().numpy() - want_a).max()
    assert err_a <= tol_v * max(1.0, float(np.abs(want_v).max())) / w.K + 1e-6, f"{what}: action chunk off by {err_a:.3e}"
    return rel


def test_expert_step_fp32(U):
    """Two layers in fp32 (plain kernels throughout): the chain agrees with the double-precision chain to fp32 rounding."""
    w = synth.CONFIGS["cfg1"].with_(B=2, L=2)
    _expert_case(U, w, 256, 2e-5, "expert fp32")


def test_expert_step_bf16(U):
    """Two layers at the action-expert widths in bf16 (tensor-core kernels, bf16 residual stream): a few roundings per layer
    accumulate; the velocity stays within 2 % of the double-precision chain."""
    w = synth.CONFIGS["cfg2"].with_(B=2, L=2, S=200, S_max=208)
    _expert_case(U, w, 1024, 2e-2, "expert bf16")


def test_expert_step_bf16_batched(U):
    """The same two-layer step for 64 streams (3200 rows: the 256-row tiles of every projection kernel, the two-CTA attention
    in its batched form), three streams compared."""
    w = synth.CONFIGS["cfg4"].with_(L=2, S=200, S_max=208)
    _expert_case(U, w, 1024, 2e-2, "expert bf16, 64 streams", streams=[0, 31, 63])


@pytest.mark.parametrize("B", [1, 2])
def test_norm_qkv_and_swiglu_few_rows(U, B):
    """One or two streams of 50 rows (at most 128 rows in all): the kernel with the weights as the A operand, 64 or 128
    row columns; Q/K/V routing with 20 feature tiles, SwiGLU with ragged hidden width."""
    w = synth.CONFIGS["cfg2"].with_(B=B)
    _norm_qkv_case(U, w, 0, f"norm+qkv {B * w.T} rows")
    _norm_swiglu_case(U, w, 1024, 0, f"norm+swiglu {B * w.T} rows")
    w2 = synth.CONFIGS["cfg2"].with_(B=B, Hq=3, Hkv=1, d=64, D=192)
    _norm_qkv_case(U, w2, 0, f"norm+qkv {B * w.T} rows, 320 features")
    _norm_swiglu_case(U, w2, 328, 0, f"norm+swiglu {B * w.T} rows, 328 hidden features")


def test_bounded_wait_reports_and_context_survives(U):
    """A device-side wait that nothing completes gives up after its limit, raises the status word and returns: the next
    status check reports REFLEX_ERR_TIMEOUT with the wait site, the CUDA context keeps working, and a cache created anew
    starts clean. (The probe is the library's own self-test kernel; nothing is hung or faulted.)"""
    import time
    rb = U.rb
    w = synth.CONFIGS["cfg2"]
    tw = U.Twin(w)
    tw.init_static([0], [w.S])
    tw.append([0], 3, 0)
    rb.reflex_cache_check_status(tw.g)                      # clean
    t0 = time.time()
    rb.reflex_cache_selftest_wait_limit(tw.g, 2000)         # 2 ms
    with pytest.raises(rb.ReflexError) as e:
        rb.reflex_cache_check_status(tw.g)
    assert e.value.code == rb.ERR_TIMEOUT and "wait site 127" in str(e.value)
    assert time.time() - t0 < 5.0
    with pytest.raises(rb.ReflexError):
        rb.reflex_cache_selftest_wait_limit(tw.g, 0)
    # the context is alive: a fresh cache over new memory computes correctly and reports a clear status
    tw2 = U.Twin(w)
    tw2.init_static([0], [w.S])
    tw2.append([0], 3, 0)
    tw2.attention(0, 0, what="after a reported timeout")
