"""CPU tests of the benchmark's host logic: the multi-rank aggregation (gloo, world size 2), the roofline
arithmetic and the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2607_14695_b200 import multi
    ms = [10.0 + 5.0 * rank, 100.0 - rank]          # rank 1 is slower on the first, rank 0 on the second
    dist.barrier()
    out = multi.max_over_ranks(ms)
    q.put((rank, out, multi.replica_throughput(200, world, out[0])))
    dist.destroy_process_group()


def test_max_over_ranks_and_replica_throughput_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, out, value in res:
        assert out == [15.0, 100.0]                                   # the slowest rank sets the time on every rank
        assert abs(value - 2 * 200 / 0.015) < 1e-6                    # both replicas' steps over the slowest time


def test_single_process_is_identity():
    from paper_2607_14695_b200 import multi
    assert multi.max_over_ranks([3.5, 7.0]) == [3.5, 7.0]
    assert multi.replica_throughput(50, 1, 25.0) == 2000.0


def test_algorithmic_bytes_match_the_scope_table():
    """Per (stream, layer, step): KV read 919 552 B, Q read + O write 409 600 B, attention 367.8 MFLOP (batched config)."""
    from paper_2607_14695_b200 import synth
    w = synth.CONFIGS["cfg4"]
    kv = (w.S + w.N + w.T) * w.Hkv * w.d * 2 * 2
    assert kv == 919552 and 2 * w.T * w.Hq * w.d * 2 == 409600
    assert 4 * w.T * w.Hq * (w.S + w.N + w.T) * w.d == 367820800
    w5 = synth.CONFIGS["cfg5"]
    assert (w5.S + w5.N + w5.T) * w5.Hkv * w5.d * 2 * 2 == 4573184


def test_reference_arm_prints_one_json_line():
    """`bench.py --impl reference` runs the oracle on a bounded sample on the host cores (no GPU needed)."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg2", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "denoising_steps_per_s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    # rank != 0 prints nothing and exits 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg2", "--steps", "1"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_roofline_picks_the_binding_roof_and_both_arms_print_the_same_config():
    """cfg4's attention launch: 85.07 MB and 23.54 GFLOP; at the measured peaks the tensor floor (17.4 us sustained) is above
    the HBM floor (13.2 us), so the bound is the tensor pipe and frac = tensor floor / measured; a copy-like launch is HBM-bound."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_mod", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    from paper_2607_14695_b200 import synth
    w = synth.CONFIGS["cfg4"]
    alg = bench.algorithmic_work(w)
    assert alg["attn_bytes_per_launch"] == 85065728 and abs(alg["attn_flops_per_launch"] - 23.5405e9) < 1e7
    peaks = {"hbm_gbs": 6459.3, "bf16_tflops": 1635.6, "bf16_tflops_sustained": 1354.9, "source": "measured"}
    r = bench.roofline_of(alg["attn_flops_per_launch"], alg["attn_bytes_per_launch"], 30e-6, peaks, "sustained")
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and abs(r["frac"] - 17.374e-6 / 30e-6) < 1e-3
    assert abs(r["frac_hbm"] - 85065728 / 30e-6 / 1e9 / 6459.3) < 1e-9 and abs(r["achieved"] - 784.7) < 0.1
    r2 = bench.roofline_of(1e6, 13.8e6, 4.5e-6, peaks, "burst")
    assert r2["bound"] == "hbm" and r2["unit"] == "GB/s" and abs(r2["frac"] - r2["frac_hbm"]) < 1e-12
    cfg = bench.config_of(w)
    assert cfg["workload"].startswith("cfg4:") and "larger than L2" in cfg["l2_policy"] and cfg["flops_per_step"] == 18 * alg["attn_flops_per_launch"]
    assert "flushed" in bench.config_of(synth.CONFIGS["cfg2"])["l2_policy"]
    traffic, src = bench.ncu_traffic(w, "auto")
    assert traffic and traffic < alg["attn_bytes_per_launch"] and "profiles/" in src
