"""Oracle for the overlap scheduler. TEST INFRASTRUCTURE ONLY: nothing in the product path may import this file.

Algorithm 1 (future-conditional overlap scheduling; Sec. 3.4 "Stream Throughput: Asynchronous Pipeline") taken step by
step in the paper's order and notation, in continuous time: one iteration of the inner loop lasts one control period
tau_step. Readings where the paper is silent (the same as the library's header states): the mean inference latency is the
arithmetic mean of the last 8 measurements, the initial estimate before the first; K is clamped to [0, C - 1]."""
import math
from fractions import Fraction


def lookahead(latencies, tau_inf_init, tau_step, C):
    """Line 3: K <- ceil(mean tau_inf / tau_step)."""
    window = latencies[-8:]
    mean = sum(window) / len(window) if window else tau_inf_init
    K = math.ceil(mean / tau_step - 1e-12)
    return max(0, min(C - 1, K))


def run(C, tau_step, tau_inf_init, tau_inf, mode="adaptive", fixed_K=0):
    """Executes len(tau_inf) chunks. Returns per-chunk records (K, launch time, ready time, stall) and totals."""
    t = 0.0                      # queue <- initial_inference(): the clock starts when the first chunk is available
    measured = []
    chunks = []
    for c, tau in enumerate(tau_inf):            # while not done
        K = lookahead(measured, tau_inf_init, tau_step, C) if mode == "adaptive" else (0 if mode == "sync" else max(0, min(C - 1, fixed_K)))
        t0 = t
        t_launch = None
        for i in range(1, C + 1):                # for i = 1 to C
            t += tau_step                        #   execute queue.pop(): one control period
            if mode != "sync" and i == C - K:    #   if i = C - K: predict the future state, launch the next inference
                t_launch = t
        if mode == "sync":
            t_launch = t                         # synchronous baseline: perceive and infer only after the chunk has ended
        t_ready = t_launch + tau
        stall = max(0.0, t_ready - t)            # queue <- await(next_chunk)
        chunks.append({"K": K, "t0": t0, "t_launch": t_launch, "t_ready": t_ready, "stall": stall,
                       "stall_ticks": math.ceil(stall / tau_step - 1e-9), "staleness": (t + stall) - t_launch})
        t += stall
        measured.append(tau)
    return {"chunks": chunks, "total_time": t, "stall_time": sum(ch["stall"] for ch in chunks),
            "stall_ticks": sum(ch["stall_ticks"] for ch in chunks),
            "mean_staleness": sum(ch["staleness"] for ch in chunks) / len(chunks),
            "mean_lookahead": sum(ch["K"] for ch in chunks) / len(chunks)}


def run_exact(C, tau_step, tau_inf_init, tau_inf):
    """The adaptive run in exact rational arithmetic (inputs as Fractions): total stall time without rounding."""
    t = Fraction(0)
    measured = []
    stall_total = Fraction(0)
    for tau in tau_inf:
        window = measured[-8:]
        mean = sum(window, Fraction(0)) / len(window) if window else tau_inf_init
        K = max(0, min(C - 1, math.ceil(mean / tau_step)))
        t_launch = t + (C - K) * tau_step
        t_end = t + C * tau_step
        stall = max(Fraction(0), t_launch + tau - t_end)
        stall_total += stall
        t = t_end + stall
        measured.append(tau)
    return stall_total, t
