#!/usr/bin/env python
"""Benchmark of the Reflex hot path on B200: denoising steps/s over one batch of synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg4] [--impl ours|reference]
    python bench.py --config frames --frames 10 --T 50 --streams 16      # ablation shapes: context window / chunk length

A "step" is one pass of the whole hot path: for each of the L layers AdaRMSNorm then partitioned
attention, then the Euler update, over all B streams (inputs resident in HBM). Prints ONE JSON line.
With N > 1 (torchrun) every rank runs an independent replica on its own GPU: the path has no exchange
step, so there is no data-path collective; the reported time is the max over ranks.

Besides the headline (`value`, `ms_per_step`: exactly K steps after W warm-up steps) the line carries
  regimes     the step and the attention launch in both SM-clock regimes of this part (a burst of a few ms at the maximum
              clock; a run of >= 2 s, which settles under the power cap), each with the SM clock sampled during the leg
              and the duration in SM cycles (time x median MHz), so that no figure depends on --steps
  roofline    the attention kernel against its binding roof (tensor pipe or HBM, whichever floor is higher), sustained
              leg against the sustained peak, burst leg against the burst peak, the HBM fraction beside it
  chained_step   the step whose layers run AdaRMSNorm + packed Q/K/V projection -> attention, with its own roofline
  extra       (default run only) the batch-1 stream of cfg3: per-tick latency over 50 ticks; the long-context attention of cfg5;
              the whole expert step at 1, 4 and 16 streams
  e2e, e2e_expert   end to end from pinned host buffers: per-layer inputs of the path; and a whole expert step, where
              only the action chunk and the conditioning vectors cross PCIe
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
L2_BYTES = 126e6


def workload_name(w):
    """The one description of a workload that both arms print in `config.workload`."""
    return (f"{w.name}: B={w.B} streams x L={w.L} layers, Hq={w.Hq}/Hkv={w.Hkv}, d={w.d}, static S={w.S}, ring N={w.N}, "
            f"dynamic T={w.T}, D={w.D}, K={w.K}; one step = L x (AdaRMSNorm + partitioned attention) + Euler update")


def algorithmic_work(w):
    """Bytes and FLOPs the method must move / compute (the per-unit figures of the scope table times the units of a launch)."""
    from paper_2607_14695_b200 import synth
    es = 2 if w.dtype == synth.DTYPE_BF16 else 4
    kv = (w.S + w.N + w.T) * w.Hkv * w.d * es * 2
    qo = 2 * w.T * w.Hq * w.d * es
    attn_bytes = w.B * (kv + qo)
    norm_bytes = w.B * (2 * w.T * w.D * es + w.Cd * es) + (w.Hd * w.Cd + w.D * w.Hd + w.Hd + w.D) * es
    flow_bytes = w.B * w.T * w.A * (8 + es)
    attn_flops = 4.0 * w.B * w.T * w.Hq * (w.S + w.N + w.T) * w.d
    n_out = (w.Hq + 2 * w.Hkv) * w.d
    qkv_flops = 2.0 * w.B * w.T * w.D * n_out
    qkv_bytes = (w.B * w.T * w.D + n_out * w.D + w.B * w.T * n_out) * es + w.B * w.D * 4
    return {"attn_bytes_per_launch": attn_bytes, "norm_bytes_per_launch": norm_bytes, "flow_bytes_per_launch": flow_bytes,
            "bytes_per_step": w.L * (attn_bytes + norm_bytes) + flow_bytes, "attn_flops_per_launch": attn_flops,
            "flops_per_step": w.L * attn_flops, "qkv_flops_per_launch": qkv_flops, "qkv_bytes_per_launch": qkv_bytes}


def resident_input_bytes(w, variants=2):
    from paper_2607_14695_b200 import synth
    es = 2 if w.dtype == synth.DTYPE_BF16 else 4
    per_layer = w.B * w.T * (w.D + w.Hq * w.d + 2 * w.Hkv * w.d) * es
    cache = 2 * w.L * w.B * (w.S_max + w.N) * w.Hkv * w.d * es
    return w.L * variants * per_layer + cache


def config_of(w):
    """`config` of the JSON line, identical in both arms (it names the workload, not how an arm runs it)."""
    alg = algorithmic_work(w)
    res = resident_input_bytes(w)
    l2 = (f"inputs larger than L2: {res / 1e6:.0f} MB of cache + per-layer inputs are read per step pair (L2 is 126 MB)" if res >= 4 * L2_BYTES
          else "L2 flushed (256 MB write) before every timed step; each step timed by its own event pair")
    return {"workload": workload_name(w), "l2_policy": l2 + " [GPU arm; the CPU arm has no such cache to defeat]",
            "bytes_per_step_algorithmic": alg["bytes_per_step"], "flops_per_step": alg["flops_per_step"]}


def make_workload(args):
    from paper_2607_14695_b200 import synth
    if args.config != "frames":
        return synth.CONFIGS[args.config]
    # the paper's ablation shapes: a sliding window of `frames` frames x 256 tokens fed one frame per tick, chunks of T tokens
    base = synth.CONFIGS["cfg4"]
    return base.with_(name=f"frames{args.frames}_T{args.T}_B{args.streams}", seed=40 + args.frames, B=args.streams, N=256 * args.frames, T=args.T, m=256)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", FALLBACK_BF16_TFLOPS)),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 1400.0)), "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def ncu_traffic(w, attn):
    """dram read + write bytes of one attention launch from the committed ncu capture (profiles/ncu_traffic.json)."""
    try:
        table = json.load(open(os.path.join(ROOT, "profiles", "ncu_traffic.json")))
    except Exception:
        return None, None
    for e in table.get("captures", []):
        if e.get("workload") == w.name and attn in e.get("attention_impl", []):
            return float(e["dram_bytes_per_launch"]), f"profiles/{e['summary']} (dram read + write of one launch, kernel source at commit {e['commit']})"
    return None, None


class ClockSampler(threading.Thread):
    """Reads (never sets) SM clock, power and clock-event reasons through NVML while the timed regions run."""

    NAMES = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
             0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples = []          # (wall time, sm_mhz, reasons bitmask, power W)
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False

    def run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
            self.ok = True
            while not self._stop_evt.is_set():
                try:
                    mhz = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
                    try:
                        reasons = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                    except Exception:
                        reasons = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                    try:
                        power = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
                    except Exception:
                        power = None
                    self.samples.append((time.time(), mhz, int(reasons), power))
                except Exception:
                    pass
                time.sleep(self.period)
        except Exception:
            self.ok = False

    def stop(self):
        self._stop_evt.set()

    def window(self, t0: float, t1: float):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        if not inside and self.samples:     # a leg shorter than the sampling period: the sample nearest to it
            mid = 0.5 * (t0 + t1)
            inside = [min(self.samples, key=lambda s: abs(s[0] - mid))]
        return inside

    def median_mhz(self, t0: float, t1: float):
        inside = self.window(t0, t1)
        return float(statistics.median(s[1] for s in inside)) if inside else None

    def summary(self, t0: float, t1: float):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = "sampled during the timed region"
        if not inside:
            inside, note = self.samples, "timed region shorter than the sampling period: samples span warm-up and timed region"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "note": "NVML unavailable"}
        mask = 0
        for s in inside:
            mask |= s[2]
        powers = [s[3] for s in inside if s[3] is not None]
        return {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.max_mhz,
                "reasons": [n for bit, n in self.NAMES.items() if mask & bit], "samples": len(inside),
                "power_w_max": max(powers) if powers else None, "note": note}


def oracle_sample_seconds(w, n_units: int):
    """Times the CPU oracle, as it stands, on n_units (stream, layer) units of the workload:
    AdaRMSNorm + attention by definition over the gathered context, plus one Euler update of the batch."""
    import numpy as np

    from oracle import reflex_oracle as orc
    from paper_2607_14695_b200 import synth

    B = min(w.B, max(1, n_units))
    L = (n_units + B - 1) // B
    wl = w.with_(B=B, L=L)
    oc = orc.OracleCache(L, B, w.Hkv, w.d, w.S_max, w.N, head0=list(synth.ring_head0(wl)))
    for b in range(B):
        oc.init_static(b, synth.normal(wl, "k_static", (L, w.S, w.Hkv, w.d), 0, b), synth.normal(wl, "v_static", (L, w.S, w.Hkv, w.d), 0, b))
        oc.append_sliding(b, synth.normal(wl, "k_new", (L, w.N, w.Hkv, w.d), 0, b), synth.normal(wl, "v_new", (L, w.N, w.Hkv, w.d), 0, b))
    x = synth.norm_input(wl, 0, 0); cond = synth.cond_vectors(wl, 1.0)
    W1, b1, W2, b2 = synth.gate_weights(wl, 0)
    q = synth.normal(wl, "q", (B, w.T, w.Hq, w.d)); kd = synth.normal(wl, "k_dyn", (B, w.T, w.Hkv, w.d)); vd = synth.normal(wl, "v_dyn", (B, w.T, w.Hkv, w.d))
    xa = synth.normal(wl, "noise", (B, w.T, w.A)).astype(np.float64); v = synth.normal(wl, "v_flow", (B, w.T, w.A))
    done = 0
    t0 = time.perf_counter()
    for layer in range(L):
        for b in range(B):
            if done >= n_units:
                break
            orc.adarmsnorm(x[b], cond[b], W1, b1, W2, b2, 1e-6)
            oc.attention(b, layer, q[b], kd[b], vd[b])
            done += 1
    orc.flow_step(xa, v, w.K)
    return time.perf_counter() - t0, orc.max_threads()


def run_reference(args, w):
    """The reference arm is the CPU oracle (there is no other implementation of the paper's method here):
    each step is a bounded sample of the workload, scaled to a whole step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    units = w.B * w.L
    t1, threads = oracle_sample_seconds(w, 1)
    budget = 100.0 / max(1, args.steps + args.warmup)
    n = int(max(1, min(units, budget / max(t1, 1e-6))))
    for _ in range(args.warmup):
        oracle_sample_seconds(w, n)
    times = [oracle_sample_seconds(w, n)[0] for _ in range(args.steps)]
    sec_per_step = statistics.mean(times) * units / n
    value = 1.0 / sec_per_step
    sample = f"{n} of {units} (stream, layer) units per step (AdaRMSNorm + attention by definition) + one Euler update, scaled by {units}/{n}"
    line = {"impl": "reference", "metric": "denoising_steps_per_s", "value": value, "unit": "steps/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w),
            "run": {"sampled": True, "seconds_per_sampled_step": statistics.mean(times),
                    "note": "ms_per_step is the sampled time scaled to a whole step: the run itself lasts (steps + warmup) x seconds_per_sampled_step"},
            "cpu_baseline": {"value": value, "unit": "steps/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def roofline_of(flops, nbytes, seconds, peaks, regime):
    """A launch (or step) against its binding roof: the higher of the HBM floor (measured copy bandwidth) and the tensor floor
    (measured cuBLAS bf16 rate: burst figure for a short leg at the maximum clock, sustained figure for a long one)."""
    tf_peak = peaks["bf16_tflops"] if regime == "burst" else peaks["bf16_tflops_sustained"]
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tensor = flops / (tf_peak * 1e12)
    bound = "tensor" if t_tensor >= t_hbm else "hbm"
    gbs, tfs = nbytes / seconds / 1e9, flops / seconds / 1e12
    out = {"bound": bound, "unit": "TFLOP/s" if bound == "tensor" else "GB/s", "achieved": tfs if bound == "tensor" else gbs,
           "peak": tf_peak if bound == "tensor" else peaks["hbm_gbs"], "frac": max(t_hbm, t_tensor) / seconds,
           "frac_hbm": gbs / peaks["hbm_gbs"], "frac_tensor": tfs / tf_peak, "achieved_gbs": gbs, "achieved_tflops": tfs,
           "floor_us": {"hbm": t_hbm * 1e6, "tensor": t_tensor * 1e6}, "regime": regime, "peak_source": peaks["source"]}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg4", choices=["cfg2", "cfg3", "cfg4", "cfg5", "frames"])
    ap.add_argument("--frames", type=int, default=10, help="--config frames: frames of 256 tokens in the sliding window")
    ap.add_argument("--T", type=int, default=50, help="--config frames: action-chunk length")
    ap.add_argument("--streams", type=int, default=16, help="--config frames: streams")
    ap.add_argument("--attn", default="auto", choices=["auto", "simt", "tc", "tc2"])
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the cfg3 stream leg and the cfg5 attention leg of the default run")
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="length of the sustained-clock legs (0: skip them)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--ticks", type=int, default=500, help="ticks of the streaming trace (single-stream configs)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2607_14695_b200 import synth
    w = make_workload(args)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist

    from paper_2607_14695_b200 import binding as rb
    from paper_2607_14695_b200 import build as rbuild
    from paper_2607_14695_b200.runner import StepRunner

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        rbuild.build()
    if world > 1:
        dist.barrier()
    rb.load()

    impl = {"auto": rb.ATTN_AUTO, "simt": rb.ATTN_SIMT, "tc": rb.ATTN_TC, "tc2": rb.ATTN_TC2}[args.attn]
    runner = StepRunner(w, device=dev, attn_impl=impl, host_inputs=not args.no_e2e)
    alg = algorithmic_work(w)
    stream = torch.cuda.current_stream()
    use_graph = not args.no_graph
    if use_graph:
        runner.capture_steps()
    do_step = runner.step_graph if use_graph else runner.step
    l2_flush = None
    if resident_input_bytes(w) < 4 * L2_BYTES:
        l2_flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # small workload: flush L2 between steps

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_steps(n, step_fn):
        """n steps; device time by CUDA events on the launching stream. With an L2 flush between steps each step is
        bracketed by its own pair of events so the flush stays outside the timed region."""
        if l2_flush is None:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for k in range(n):
                step_fn(k)
            b.record(stream)
            barrier()
            return a.elapsed_time(b), None
        evs = []
        for k in range(n):
            l2_flush.fill_(k & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); step_fn(k); b.record(stream)
            evs.append((a, b))
        barrier()
        per = [a.elapsed_time(b) for a, b in evs]
        return sum(per), per

    sampler = ClockSampler(local_rank)
    sampler.start()
    t_wait = time.time()
    while not sampler.samples and sampler.is_alive() and time.time() - t_wait < 10.0:   # NVML is up before the timed region starts
        time.sleep(0.01)

    def cool():
        """Lets the part return to its burst clock before a short leg (2 s of idling bring it back)."""
        barrier()
        time.sleep(2.0)

    def leg(fn, n, per_call=1):
        """n calls of fn(i) between two events, with the SM clock sampled meanwhile. Returns (ms per unit, median MHz, wall s)."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.time()
        a.record(stream)
        for i in range(n):
            fn(i)
        b.record(stream)
        barrier()
        t1 = time.time()
        ms = a.elapsed_time(b)
        return ms / (n * per_call), sampler.median_mhz(t0, t1), ms * 1e-3

    def regime(ms_unit, mhz, seconds):
        return {"us": ms_unit * 1e3, "sm_mhz": mhz, "kcycles": (ms_unit * 1e3 * mhz / 1e3) if mhz else None, "leg_seconds": seconds}

    for k in range(args.warmup):
        do_step(k)
    barrier()
    # ---- timed region: exactly K steps ----
    launches0 = rb.reflex_kernel_launch_count()
    wall0 = time.time()
    ms_total, per_step = timed_steps(args.steps, do_step)
    wall1 = time.time()
    launches = (sum(runner.kernels_each[k % len(runner.kernels_each)] for k in range(args.steps)) if use_graph
                else (rb.reflex_kernel_launch_count() - launches0))
    clocks = sampler.summary(wall0, wall1)
    headline_mhz = sampler.median_mhz(wall0, wall1)

    # ---- the same step in both clock regimes (no L2 flush inside these legs: big workloads only) ----
    regimes = {}
    sustain = args.sustain_seconds if l2_flush is None else 0.0
    if l2_flush is None:
        cool()
        ms_u, mhz, sec = leg(do_step, 16)
        regimes["step_burst"] = regime(ms_u, mhz, sec)
        if sustain > 0:
            n_sus = max(args.steps, int(sustain / max(ms_u * 1e-3, 1e-6)))
            ms_u, mhz, sec = leg(do_step, n_sus)
            regimes["step_sustained"] = regime(ms_u, mhz, sec)

    # ---- per-kernel durations: graphs that hold only the attention (resp. AdaRMSNorm) launches of one step ----
    reps = max(3, min(args.steps, 20))

    def kernel_graphs(r, fn_variant):
        graphs = [r.capture(lambda v=v: fn_variant(v))[0] for v in range(r.variants)]
        for g in graphs:
            g.replay()
        barrier()
        return graphs

    def avg_launch_ms(fn_variant, calls_per_graph, r=runner):
        graphs = kernel_graphs(r, fn_variant)
        return leg(lambda i: graphs[i % len(graphs)].replay(), reps, calls_per_graph)[0]

    def attention_legs(r):
        """Attention launches of one step per graph, replayed in a short burst after a pause and in a long run."""
        graphs = kernel_graphs(r, lambda v: [r.attention(l, v, sh()) for l in range(r.w.L)])
        cool()
        ms_b, mhz_b, sec_b = leg(lambda i: graphs[i % len(graphs)].replay(), 6, r.w.L)
        out = {"burst": regime(ms_b, mhz_b, sec_b)}
        if args.sustain_seconds > 0:
            n_sus = max(6, int(args.sustain_seconds / max(ms_b * 1e-3 * r.w.L, 1e-6)))
            ms_s, mhz_s, sec_s = leg(lambda i: graphs[i % len(graphs)].replay(), n_sus, r.w.L)
            out["sustained"] = regime(ms_s, mhz_s, sec_s)
        return out

    sh = rb.stream_handle
    attn = attention_legs(runner)
    attn_main = attn.get("sustained", attn["burst"])
    attn_main_regime = "sustained" if "sustained" in attn else "burst"
    attn_avg_ms = attn_main["us"] * 1e-3
    regimes["attention_burst"] = attn["burst"]
    if "sustained" in attn:
        regimes["attention_sustained"] = attn["sustained"]
    regimes["note"] = ("burst: a few ms of launches after 2 s of idling (maximum SM clock); sustained: >= --sustain-seconds of back-to-back launches "
                       "(the clock the power cap settles at); kcycles = us x median sampled SM MHz / 1000: the same launch costs about the same SM cycles in both")
    norm_avg_ms = avg_launch_ms(lambda v: [runner.norm(l, v, v, sh()) for l in range(w.L)], w.L)   # the stand-alone call: gate MLP + rows
    # what the step itself launches for AdaRMSNorm: the gate MLPs of all L layers in one call (two kernels), then one rows kernel per layer
    gates_step_ms = avg_launch_ms(lambda v: runner.gates_of_step(v, sh()), 1)
    gates_tick_ms = avg_launch_ms(lambda v: runner.gates_of_tick(sh()), 1)   # what the steps launch: once per tick of K steps, for all K
    rows_avg_ms = avg_launch_ms(lambda v: [runner.rows(l, v, sh(), True) for l in range(w.L)], w.L)

    # ---- the chained layer (AdaRMSNorm folded into the packed Q/K/V projection -> attention) and the whole expert step ----
    peaks = measured_peaks()
    chained, chained_step, e2e_expert = None, None, None
    if runner.tdt == torch.bfloat16:
        from paper_2607_14695_b200 import expert as ex
        F = 4 * w.D
        qkv_avg_ms = avg_launch_ms(lambda v: [runner.norm_qkv(l, v, sh()) for l in range(w.L)], w.L)
        swiglu_avg_ms = avg_launch_ms(lambda v: [runner.norm_swiglu(l, v, sh()) for l in range(w.L)], w.L)
        cgraphs = kernel_graphs(runner, lambda v: runner.step_chained(v))
        chained_ms, chained_mhz, chained_sec = leg(lambda i: cgraphs[i % len(cgraphs)].replay(), max(reps, int(0.5 * sustain / 1e-3) if sustain > 0 else reps))
        ch_flops = w.L * (alg["qkv_flops_per_launch"] + alg["attn_flops_per_launch"])
        # x and W_QKV in, Q / K_dyn / V_dyn written and read back, the cached K / V, O out
        ch_bytes = w.L * (alg["qkv_bytes_per_launch"] + alg["attn_bytes_per_launch"]) + alg["flow_bytes_per_launch"]
        chained_step = {"ms_per_step": chained_ms, "steps_per_s": 1e3 / chained_ms, "sm_mhz": chained_mhz, "leg_seconds": chained_sec,
                        "flops_per_step": ch_flops, "bytes_per_step_algorithmic": ch_bytes,
                        "roofline": roofline_of(ch_flops, ch_bytes, chained_ms * 1e-3, peaks, "sustained" if chained_sec >= 0.5 else "burst"),
                        "what": "gates of the step (one call), then per layer AdaRMSNorm + packed W_QKV projection in one launch and the partitioned attention over its "
                                "Q / K_dyn / V_dyn, then the Euler update: 2 L + 3 launches, no stand-alone norm launch"}
        # a whole action-expert step: the fused calls, the output / down projections with residual and the two A-wide heads (reflex_linear_residual)
        model = ex.ActionExpert(w, runner.cache, ex.random_weights_device(w, F, device=dev), F, device=dev)
        # (both clock regimes, like the headline: what ran just before this leg would otherwise decide which one it lands in)
        ex_graphs = kernel_graphs(runner, lambda v: model.step(runner.xa, runner.cond[v % w.K], v % w.K))
        cool()
        ex_b = leg(lambda i: ex_graphs[i % len(ex_graphs)].replay(), 6, 1)
        expert_ms = ex_b[0]
        expert_regimes = {"burst": regime(*ex_b)}
        if args.sustain_seconds > 0:
            ex_s = leg(lambda i: ex_graphs[i % len(ex_graphs)].replay(), max(6, int(min(args.sustain_seconds, 1.0) / max(ex_b[0] * 1e-3, 1e-6))), 1)
            expert_regimes["sustained"] = regime(*ex_s)
        del ex_graphs
        lin = {}
        for name, Kc in (("output_projection", w.Hq * w.d), ("down_projection", F)):
            a_in = [runner.rnd(w.B * w.T, Kc) for _ in range(runner.variants)]
            Wl = [runner.rnd(w.D, Kc, std=float(Kc) ** -0.5) for _ in range(runner.variants)]
            hres = [runner.rnd(w.B * w.T, w.D) for _ in range(runner.variants)]
            calls = [rb.prepare_linear_residual(a_in[v], Wl[v], hres[v], hres[v], cache=runner.cache) for v in range(runner.variants)]
            ms_lin = avg_launch_ms(lambda v: [calls[v](sh()) for _ in range(6)], 6)
            lib_graphs = kernel_graphs(runner, lambda v: [hres[v].addmm_(a_in[v], Wl[v].t()) for _ in range(6)])
            ms_lib = leg(lambda i: lib_graphs[i % len(lib_graphs)].replay(), reps, 6)[0]
            lin[name] = {"shape_mnk": [w.B * w.T, w.D, Kc], "avg_us": ms_lin * 1e3, "tflops": 2.0 * w.B * w.T * w.D * Kc / (ms_lin * 1e-3) / 1e12,
                         "library_gemm_avg_us": ms_lib * 1e3}
            del a_in, Wl, hres, calls, lib_graphs
        n_out = (w.Hq + 2 * w.Hkv) * w.d
        chained = {"norm_qkv_avg_us": qkv_avg_ms * 1e3, "norm_qkv_tflops": alg["qkv_flops_per_launch"] / (qkv_avg_ms * 1e-3) / 1e12,
                   "norm_qkv_shape_mnk": [w.B * w.T, n_out, w.D], "ms_per_step": chained_ms,
                   "norm_swiglu_avg_us": swiglu_avg_ms * 1e3, "norm_swiglu_tflops": 2.0 * w.B * w.T * w.D * 2 * F / (swiglu_avg_ms * 1e-3) / 1e12,
                   "norm_swiglu_shape_m_f_k": [w.B * w.T, F, w.D], "linear_residual": lin, "expert_step_ms": expert_ms, "expert_step_regimes": expert_regimes,
                   "what": "norm_qkv / norm_swiglu: AdaRMSNorm folded into the packed Q/K/V projection resp. the fused gate/up projections, timed alone; "
                           "linear_residual: the output and down projections with their residual add (reflex_linear_residual) beside torch.addmm_ on the same shapes; "
                           "expert_step_ms (burst clocks; expert_step_regimes has the sustained leg too): a whole action-expert denoising step (input projection, L x (norm+QKV, attention, output projection, norm+SwiGLU, "
                           "down projection), velocity head, Euler update; F = 4 D); every contraction is this library's kernel (the two A-wide heads go through reflex_linear_residual without a residual)"}
        if not args.no_e2e:
            # end to end through the expert step: the action chunk and the conditioning vectors come from pinned host memory
            # every step and the updated chunk goes back; nothing else crosses PCIe
            h_a = torch.randn(w.B, w.T, w.A).pin_memory()
            h_c = [runner.cond[k].cpu().pin_memory() for k in range(w.K)]
            h_out = torch.empty(w.B, w.T, w.A).pin_memory()
            d_c = torch.empty_like(runner.cond[0])

            def expert_e2e(k):
                runner.xa.copy_(h_a, non_blocking=True)
                d_c.copy_(h_c[k % w.K], non_blocking=True)
                model.step(runner.xa, d_c, k % w.K)
                h_out.copy_(runner.xa, non_blocking=True)

            for k in range(3):
                expert_e2e(k)
            ms_e, _, _ = leg(expert_e2e, max(3, min(args.steps, 30)))
            e2e_expert = {"value": world * 1e3 / ms_e, "unit": "steps/s", "ms_per_step": ms_e,
                          "h2d_bytes_per_step": int(h_a.numel() * 4 + h_c[0].numel() * h_c[0].element_size()), "d2h_bytes_per_step": int(h_out.numel() * 4),
                          "what": "one whole expert step per call through the public API (ActionExpert.step, direct launches): H2D of the action chunk and the "
                                  "conditioning vectors, all kernels, D2H of the updated chunk"}
        del model

    step_marks = []
    for k in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); do_step(k); b.record(stream)
        step_marks.append((a, b))
    barrier()
    step_ms = sorted(a.elapsed_time(b) for a, b in step_marks) if per_step is None else sorted(per_step)

    # ---- end to end: inputs from pinned host memory, action chunk back to the host, every step ----
    e2e_ms = 0.0
    n_e2e = max(3, min(args.steps, 30))
    if not args.no_e2e:
        # Every step's inputs are copied from pinned host memory and its action chunk is copied back, all inside the timed
        # region. The copies run on a second stream into the input set the previous step is not using (the runner keeps two
        # sets), so the copy of step k + 1 overlaps the kernels of step k; events order both directions.
        copy_stream = torch.cuda.Stream()
        ready = [torch.cuda.Event() for _ in range(runner.variants)]
        done = [torch.cuda.Event() for _ in range(runner.variants)]

        def stage(k):
            v = k % runner.variants
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(done[v])          # the step that last read this input set has finished
                runner.copy_inputs_from_host(k)
                ready[v].record(copy_stream)

        def e2e_run(k0, n):
            copy_stream.wait_stream(stream)
            stage(k0)
            for k in range(k0, k0 + n):
                if k + 1 < k0 + n:
                    stage(k + 1)
                v = k % runner.variants
                stream.wait_event(ready[v])
                do_step(k)
                runner.copy_result_to_host()
                done[v].record(stream)

        e2e_run(0, 4)
        barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        e2e_run(4, n_e2e)
        h1.record(stream)
        barrier()
        e2e_ms = h0.elapsed_time(h1)

    def stream_trace(r, n_ticks, S_hi):
        """A streaming trace on runner r: one CUDA-graph replay per control tick, a new static prefix every 10 ticks."""
        r.capture_tick()
        ev = []
        for tck in range(n_ticks + 5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            if tck % 10 == 0:
                r.refresh_static(S_hi if (tck // 10) % 2 == 0 else S_hi - 16)   # new observation, alternating prefix length
            r.tick_graph.replay()
            b.record(stream)
            ev.append((a, b))
        barrier()
        rb.reflex_cache_check_status(r.cache)
        tms = sorted(a.elapsed_time(b) for a, b in ev[5:])
        return {"ticks": n_ticks, "steps_per_tick": r.w.K, "tick_ms_p50": tms[len(tms) // 2], "tick_ms_p95": tms[min(len(tms) - 1, int(0.95 * len(tms)))],
                "tick_ms_max": tms[-1], "budget_ms": 20.0, "sustains_50hz": tms[-1] < 20.0, "kernels_per_tick": r.kernels_per_tick,
                "note": "one tick = ring append (all layers) + noise + K steps, replayed as one CUDA graph; a new static prefix every 10 ticks; cache stays L2-resident across a tick by nature"}

    # ---- streaming trace (single-stream configs): per-tick device latency against the 50 Hz budget ----
    stream_stats = None
    if w.ticks > 1 and w.B == 1:
        n_ticks = min(w.ticks, args.ticks)
        stream_stats = stream_trace(runner, n_ticks, w.S)
        # the same trace with the asynchronous hand-over: every 10 ticks a producer stream stages the next prefix in the
        # idle static bank while ticks keep running, and the consumer flips banks at the following tick boundary
        r2 = StepRunner(w, device=dev, static_banks=2)
        r2.capture_tick()
        producer = torch.cuda.Stream()
        tick_ev2, staged = [], False
        for tck in range(n_ticks + 5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            if staged:
                stream.wait_stream(producer)
                r2.commit_static()
                staged = False
            if tck % 10 == 0:
                r2.stage_static(w.S if (tck // 10) % 2 == 0 else w.S - 16, producer)
                staged = True
            r2.tick_graph.replay()
            b.record(stream)
            tick_ev2.append((a, b))
        barrier()
        rb.reflex_cache_check_status(r2.cache)
        tms2 = sorted(a.elapsed_time(b) for a, b in tick_ev2[5:])
        stream_stats["async_prefix"] = {"tick_ms_p50": tms2[len(tms2) // 2], "tick_ms_max": tms2[-1],
                                        "note": "new prefix staged on a second stream into the idle static bank during the ticks, committed (index flip) at the next tick boundary"}
        del r2

    # ---- default run only: the two other halves of the target, so that one line carries them ----
    extra = None
    if args.config == "cfg4" and not args.no_extra and world == 1:
        extra = {}
        w3 = synth.CONFIGS["cfg3"]
        r3 = StepRunner(w3, device=dev)
        extra["cfg3_stream"] = dict(stream_trace(r3, 50, w3.S), workload=workload_name(w3))
        del r3
        w5 = synth.CONFIGS["cfg5"]
        r5 = StepRunner(w5, device=dev)
        a5 = attention_legs(r5)
        alg5 = algorithmic_work(w5)
        m5 = a5.get("sustained", a5["burst"])
        extra["cfg5_attention"] = {"workload": workload_name(w5), "regimes": a5,
                                   "roofline": roofline_of(alg5["attn_flops_per_launch"], alg5["attn_bytes_per_launch"], m5["us"] * 1e-6, peaks,
                                                           "sustained" if "sustained" in a5 else "burst"),
                                   "roofline_burst": roofline_of(alg5["attn_flops_per_launch"], alg5["attn_bytes_per_launch"], a5["burst"]["us"] * 1e-6, peaks, "burst")}
        t5, src5 = ncu_traffic(w5, args.attn)
        extra["cfg5_attention"]["roofline"].update({"traffic": t5, "traffic_source": src5, "bytes_per_launch": alg5["attn_bytes_per_launch"]})
        rb.reflex_cache_check_status(r5.cache)
        del r5
        # the whole expert step at few streams (cfg4's shapes): where serving a handful of robots sits between cfg3 and cfg4
        from paper_2607_14695_b200 import expert as ex_few
        few = {}
        for Bf in (1, 4, 16):
            wf = w.with_(B=Bf)
            rf = StepRunner(wf, device=dev)
            mf = ex_few.ActionExpert(wf, rf.cache, ex_few.random_weights_device(wf, 4 * wf.D, device=dev), 4 * wf.D, device=dev)
            gf = kernel_graphs(rf, lambda v: mf.step(rf.xa, rf.cond[v % wf.K], v % wf.K))
            cool()
            ms_f, mhz_f, _ = leg(lambda i: gf[i % len(gf)].replay(), 6, 1)
            rb.reflex_cache_check_status(rf.cache)
            few[str(Bf)] = {"expert_step_ms": ms_f, "sm_mhz": mhz_f, "us_per_layer": ms_f * 1e3 / wf.L}
            del gf, mf, rf
        extra["expert_step_by_streams"] = dict(few, what="whole action-expert step (CUDA graph, burst clocks) at 1, 4 and 16 streams of 50 tokens, cfg4's layer shapes, F = 4 D")
    sampler.stop()

    from paper_2607_14695_b200 import multi
    ms_total, e2e_ms_max = multi.max_over_ranks([ms_total, e2e_ms], device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms_total / args.steps
    value = multi.replica_throughput(args.steps, world, ms_total)     # every rank runs its own replica of the batch
    roof = roofline_of(alg["attn_flops_per_launch"], alg["attn_bytes_per_launch"], attn_avg_ms * 1e-3, peaks, attn_main_regime)
    traffic, traffic_src = ncu_traffic(w, args.attn)
    roof.update({"kernel": "partitioned attention", "traffic": traffic, "traffic_source": traffic_src,
                 "bytes_per_launch": alg["attn_bytes_per_launch"], "flops_per_launch": alg["attn_flops_per_launch"], "avg_launch_us": attn_avg_ms * 1e3,
                 "how": "graphs that hold only the L attention launches of a step, replayed back to back; CUDA events on the launching stream; "
                        "frac = max(HBM floor, tensor floor) / measured, frac_hbm = algorithmic bytes / time / measured copy bandwidth",
                 "frac_of_nominal_8TBs": roof["achieved_gbs"] / 8000.0,
                 "burst": roofline_of(alg["attn_flops_per_launch"], alg["attn_bytes_per_launch"], attn["burst"]["us"] * 1e-6, peaks, "burst")})
    line = {
        "metric": "denoising_steps_per_s", "value": value, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "us_per_step": ms_per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == synth.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": config_of(w),
        "run": {"parallelism": "replicas only (independent streams per GPU, no collective)" if world > 1 else "single GPU",
                "attention_impl": args.attn, "launch": "CUDA graph replay, one graph per step" if use_graph else "direct launches",
                "gates": "gate MLPs of all K steps and L layers once per tick of K steps (the first step of every K carries the two gate launches)",
                "timed_region_seconds": ms_total * 1e-3, "sm_mhz": headline_mhz,
                "step_kcycles": (ms_per_step * 1e3 * headline_mhz / 1e3) if headline_mhz else None},
        "gpu_launches": int(launches),
        "step_ms": {"p50": step_ms[len(step_ms) // 2], "p95": step_ms[min(len(step_ms) - 1, int(0.95 * len(step_ms)))], "max": step_ms[-1],
                    "note": "per-step event pairs"},
        "hbm_gbs_whole_step": alg["bytes_per_step"] / (ms_per_step * 1e-3) / 1e9,
        "regimes": regimes,
        "roofline": roof,
        "chained_step": chained_step,
        "chained_layer": chained,
        "kernels": {"attention_avg_us": attn_avg_ms * 1e3, "attention_burst_us": attn["burst"]["us"], "adarmsnorm_rows_avg_us": rows_avg_ms * 1e3,
                    "adarmsnorm_gates_of_step_us": gates_step_ms * 1e3, "adarmsnorm_gates_of_tick_us": gates_tick_ms * 1e3,
                    "adarmsnorm_rows_gbs": alg["norm_bytes_per_launch"] / (rows_avg_ms * 1e-3) / 1e9,
                    "adarmsnorm_rows_frac_hbm": alg["norm_bytes_per_launch"] / (rows_avg_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "adarmsnorm_standalone_call_avg_us": norm_avg_ms * 1e3,
                    "attention_share_of_step": (attn["burst"]["us"] * w.L / regimes["step_burst"]["us"]) if "step_burst" in regimes
                                               else attn["burst"]["us"] * 1e-3 * w.L / statistics.mean(step_ms)},
        "clocks": clocks,
    }
    if stream_stats is not None:
        line["stream"] = stream_stats
    if extra is not None:
        line["extra"] = extra
        line["stream"] = line.get("stream") or dict(extra["cfg3_stream"], config="cfg3 (batch-1 stream), measured in this run beside the headline workload")
    if not args.no_e2e:
        line["e2e"] = {"value": multi.replica_throughput(n_e2e, world, e2e_ms_max), "unit": "steps/s", "h2d_bytes_per_step": int(runner.h2d_bytes_per_step),
                       "d2h_bytes_per_step": int(runner.d2h_bytes_per_step), "steps": n_e2e,
                       "what": "the path's own calls: every layer's x, Q, K_dyn, V_dyn come from pinned host memory each step (PCIe-bound by construction)"}
        if e2e_expert is not None:
            line["e2e_expert"] = e2e_expert
    if world == 1 and not args.no_cpu_baseline:
        units = w.B * w.L
        t1, threads = oracle_sample_seconds(w, 1)
        n = int(max(1, min(units, args.cpu_seconds / max(t1, 1e-6))))
        ts, threads = oracle_sample_seconds(w, n)
        line["cpu_baseline"] = {"value": 1.0 / (ts * units / n), "unit": "steps/s", "cores": threads, "kind": "oracle",
                                "sample": f"{n} of {units} (stream, layer) units (AdaRMSNorm + attention by definition) + one Euler update, "
                                          f"{ts:.1f} s of CPU time, scaled by {units}/{n}"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
