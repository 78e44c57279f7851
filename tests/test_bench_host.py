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
