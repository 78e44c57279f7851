"""Algorithm 1 (future-conditional overlap scheduling, Sec. 3.4): pins of the oracle and parity of the library's host code
with it. No GPU work: the library is loaded for its host functions only."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import overlap_oracle as oo
from paper_2607_14695_b200 import binding as rb
from paper_2607_14695_b200 import build as rbuild


@pytest.fixture(scope="module", autouse=True)
def _lib():
    rbuild.build()


# ---- pins of the oracle: closed forms ----

def test_constant_latency_closed_forms():
    """tau_inf constant: K = ceil(tau_inf / tau_step). Overlapped: no stall once K tau_step >= tau_inf, i.e. always after the
    first chunk (whose K comes from the initial estimate); synchronous: every chunk stalls exactly tau_inf. The paper's
    setting: C = 50 actions at 50 Hz, inference of 87 ms -> K = 5."""
    C, step, tau = 50, 0.02, 0.087
    r = oo.run(C, step, 0.0, [tau] * 20)
    assert [ch["K"] for ch in r["chunks"]] == [0] + [5] * 19
    assert abs(r["chunks"][0]["stall"] - tau) < 1e-12 and all(ch["stall"] == 0.0 for ch in r["chunks"][1:])
    assert all(abs(ch["staleness"] - 5 * step) < 1e-12 for ch in r["chunks"][1:])
    s = oo.run(C, step, 0.0, [tau] * 20, mode="sync")
    assert abs(s["stall_time"] - 20 * tau) < 1e-9 and s["stall_ticks"] == 20 * 5
    assert abs(s["total_time"] - 20 * (C * step + tau)) < 1e-9
    assert abs(r["total_time"] - (20 * C * step + tau)) < 1e-9


def test_fixed_lookahead_stall_formula():
    """Fixed K: stall per chunk = max(0, tau_inf - K tau_step) exactly."""
    C, step = 10, 0.05
    taus = [0.01, 0.12, 0.26, 0.05, 0.49]
    for K in (0, 1, 3, 9):
        r = oo.run(C, step, 0.0, taus, mode="fixed", fixed_K=K)
        for ch, tau in zip(r["chunks"], taus):
            assert abs(ch["stall"] - max(0.0, tau - K * step)) < 1e-12


def test_exact_rational_run_agrees():
    rng = np.random.default_rng(0)
    taus = [Fraction(int(v), 1000) for v in rng.integers(20, 400, size=40)]
    stall, total = oo.run_exact(20, Fraction(1, 50), Fraction(1, 10), taus)
    r = oo.run(20, 0.02, 0.1, [float(t) for t in taus])
    assert abs(r["stall_time"] - float(stall)) < 1e-9 and abs(r["total_time"] - float(total)) < 1e-9


def test_lookahead_clamps_and_window():
    assert oo.lookahead([], 0.1, 0.02, 50) == 5
    assert oo.lookahead([], 5.0, 0.02, 50) == 49              # never more than C - 1
    assert oo.lookahead([0.0] * 3, 0.1, 0.02, 50) == 0
    assert oo.lookahead([1.0] * 8 + [0.02] * 8, 0.1, 0.02, 50) == 1   # only the last 8 measurements count
    assert oo.lookahead([0.04], 0.1, 0.02, 50) == 2                   # an exact multiple is not rounded up


# ---- the library against the oracle ----

@pytest.mark.parametrize("mode,name", [(0, "adaptive"), (1, "sync"), (2, "fixed")])
def test_simulate_matches_oracle(mode, name):
    rng = np.random.default_rng(11 + mode)
    for trial in range(20):
        C = int(rng.integers(1, 60))
        step = float(rng.choice([0.01, 0.02, 0.05]))
        n = int(rng.integers(1, 80))
        taus = list(rng.gamma(2.0, 0.03, size=n)) if trial % 2 else list(rng.choice([0.0, 0.02, 0.04, 0.1, 0.33], size=n))
        init = float(rng.choice([0.0, 0.05, 2.0]))
        K = int(rng.integers(0, 70))
        want = oo.run(C, step, init, taus, mode=name, fixed_K=K)
        got = rb.reflex_overlap_simulate(C, step, init, taus, mode=mode, fixed_K=K)
        assert got["chunks"] == n and got["stall_ticks"] == want["stall_ticks"]
        assert abs(got["stall_time_s"] - want["stall_time"]) <= 1e-9 and abs(got["total_time_s"] - want["total_time"]) <= 1e-9
        assert abs(got["mean_staleness_s"] - want["mean_staleness"]) <= 1e-9 and abs(got["mean_lookahead"] - want["mean_lookahead"]) <= 1e-12
        assert got["min_lookahead"] == min(ch["K"] for ch in want["chunks"]) and got["max_lookahead"] == max(ch["K"] for ch in want["chunks"])


def test_state_machine_follows_algorithm_1():
    """Drive the tick interface with a latency trace in units of control periods: the inference launched on the tick of action
    C - K completes `lat` ticks later. Launch positions, lookaheads and stall counts must match the oracle run with
    tau_step = 1 (a launch on the tick of action C - K has K whole periods plus the current one: ready by the end of the
    chunk iff lat <= K + 1, so the oracle is run with latencies lat - 1)."""
    rng = np.random.default_rng(5)
    C = 12
    lats = [int(v) for v in rng.integers(1, 9, size=30)]
    sched = rb.OverlapScheduler(C, 1.0, 3.0)
    pending = None          # ticks until the inference in flight completes
    launches, ks, stalls = [], [], 0
    chunk_seen, n_done = -1, 0
    tick = 0
    while n_done < len(lats) and tick < 10000:
        if pending is not None:
            pending -= 1
            if pending <= 0:
                sched.inference_done(float(lats[n_done]))
                n_done += 1
                pending = None
        ev = sched.tick()
        tick += 1
        if ev["stalled"]:
            stalls += 1
            continue
        if ev["chunk"] != chunk_seen:
            chunk_seen = ev["chunk"]
            ks.append(ev["lookahead"])
            assert ev["action"] == 0
        if ev["launch_now"]:
            launches.append((ev["chunk"], ev["action"]))
            pending = lats[n_done]
    want = oo.run(C, 1.0, 3.0, [float(l) for l in lats])
    assert ks[: len(lats)] == [ch["K"] for ch in want["chunks"]][: len(ks)]
    for (chunk, action), ch in zip(launches, want["chunks"]):
        assert action + 1 == C - ch["K"]                      # line 6: i = C - K (1-based)
    want_stalls = sum(max(0, l - 1 - ch["K"]) for l, ch in zip(lats, want["chunks"]))   # one period less than the end-of-period launch
    assert stalls == want_stalls


def test_error_paths():
    with pytest.raises(rb.ReflexError) as e:
        rb.OverlapScheduler(0, 0.02, 0.1)
    assert e.value.code == rb.ERR_INVALID_ARG
    s = rb.OverlapScheduler(4, 0.02, 0.1)
    with pytest.raises(rb.ReflexError) as e:
        s.inference_done(0.01)          # nothing in flight
    assert e.value.code == rb.ERR_STATE
    with pytest.raises(rb.ReflexError):
        rb.reflex_overlap_simulate(4, 0.02, 0.0, [0.1, float("nan")])
