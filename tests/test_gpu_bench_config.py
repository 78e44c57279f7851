"""Parity at the benchmark's full sizes and in its launch configuration (CUDA-graph replay of whole steps, automatic
kernel selection, gate overlap on a second stream): sampled outputs against the oracle, which reads back exactly the
bytes the kernels saw (cache slabs, ring state, per-layer inputs)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2607_14695_b200 import synth  # noqa: E402


def _oracle_for_stream(runner, layer, b):
    """Oracle cache of one (layer, stream) rebuilt from the device slab and ring state."""
    from oracle import reflex_oracle as orc
    from paper_2607_14695_b200 import binding as rb
    w = runner.w
    sl, hd, ct, _ = rb.reflex_cache_get_state(runner.cache)
    oc = orc.OracleCache(1, 1, w.Hkv, w.d, w.S_max, w.N, head0=[0])
    ks = runner.cache.k_slab[layer, b].float().cpu().numpy()
    vs = runner.cache.v_slab[layer, b].float().cpu().numpy()
    oc.k_static[0, 0] = ks[: w.S_max]; oc.v_static[0, 0] = vs[: w.S_max]
    oc.k_ring[0, 0] = ks[w.S_max:]; oc.v_ring[0, 0] = vs[w.S_max:]
    oc.static_len[0], oc.head[0], oc.count[0] = sl[b], hd[b], ct[b]
    return oc


@pytest.mark.parametrize("cfg,streams", [("cfg4", [0, 31, 63]), ("cfg5", [5])])
def test_full_size_step_graph_sampled_outputs(cfg, streams):
    from paper_2607_14695_b200 import build as rbuild
    rbuild.build()
    import gpu_util as U
    from oracle import reflex_oracle as orc
    from paper_2607_14695_b200 import binding as rb
    from paper_2607_14695_b200.runner import StepRunner

    w = synth.CONFIGS[cfg]
    runner = StepRunner(w, device=U.DEV)            # as bench.py builds it: automatic kernel choice, gate overlap
    runner.capture_steps()
    x0 = runner.xa.clone()
    for k in range(3):
        runner.step_graph(k)
    torch.cuda.synchronize()
    rb.reflex_cache_check_status(runner.cache)
    k_last, variant, layer = 2, 2 % runner.variants, w.L - 1
    # the shared y / out buffers hold the last layer of the last replayed step
    got_out = runner.out.float().cpu().numpy().astype(np.float64)
    got_y = runner.y.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got_out).all() and np.isfinite(got_y).all()
    f = lambda t: t.float().cpu().numpy()
    W1, b1, W2, b2 = [f(t) for t in runner.W[layer]]
    cond = f(runner.cond[k_last % w.K])
    for b in streams:
        oc = _oracle_for_stream(runner, layer, b)
        want = oc.attention(0, 0, f(runner.q[layer][variant][b]), f(runner.kd[layer][variant][b]), f(runner.vd[layer][variant][b]))
        U.check_close(got_out[b], want, w.dtype, f"{cfg} attention layer {layer} stream {b}")
        want_y = orc.adarmsnorm(f(runner.x[layer][variant][b]), cond[b], W1, b1, W2, b2, 1e-6)
        U.check_close(got_y[b], want_y, w.dtype, f"{cfg} norm layer {layer} stream {b}", rel_clause=True)
    # the Euler chain over the three replayed steps
    xo = x0.cpu().numpy().astype(np.float64)
    for k in range(3):
        orc.flow_step(xo, f(runner.vflow[k % runner.variants]), w.K)
    U.check_close(runner.xa.cpu().numpy().astype(np.float64), xo, synth.DTYPE_F32, f"{cfg} action chunk")
    # a middle layer through direct calls on the same runner (no graph)
    mid = w.L // 2
    sh = rb.stream_handle()
    runner.gate(mid, 0, sh); runner.rows(mid, 0, sh); runner.attention(mid, 0, sh)
    torch.cuda.synchronize()
    b = streams[0]
    oc = _oracle_for_stream(runner, mid, b)
    want = oc.attention(0, 0, f(runner.q[mid][0][b]), f(runner.kd[mid][0][b]), f(runner.vd[mid][0][b]))
    U.check_close(runner.out[b].float().cpu().numpy().astype(np.float64), want, w.dtype, f"{cfg} attention layer {mid} direct")


def test_fused_projections_at_bench_size():
    """The two fused projections at the size and launch configuration `bench.py` times them (64 streams x 50 rows, D = 1024,
    2560 Q/K/V features in 512-column tiles; F = 4096 hidden features), compared on a sample of streams."""
    from paper_2607_14695_b200 import build as rbuild
    rbuild.build()
    import gpu_util as U
    import test_gpu_parity as tp
    w = synth.CONFIGS["cfg4"]
    tp._norm_qkv_case(U, w, 0, "bench-size norm+qkv", streams=[0, 17, 63])
    tp._norm_swiglu_case(U, w, 4 * w.D, 0, "bench-size norm+swiglu", streams=[5, 40])
    # the output and down projections at the same size (3200 rows onto D = 1024 from 2048 and 4096), a sample of rows
    rows = [0, 255, 256, 1700, 3071, 3072, 3199]
    tp._linear_case(U, w.dtype, w.B * w.T, w.Hq * w.d, w.D, 0, "bench-size output projection", in_place=True, rows=rows)
    tp._linear_case(U, w.dtype, w.B * w.T, 4 * w.D, w.D, 0, "bench-size down projection", in_place=True, rows=rows)
