"""The hand-worked fixtures of tests/golden/ (derived from the paper's equations, see the README there) against the oracle."""
import json
import os

import numpy as np

from oracle import reflex_oracle as orc

G = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
load = lambda name: json.load(open(os.path.join(G, name)))


def test_eq2_adarmsnorm_hand_cases():
    g = load("eq2_adarmsnorm_hand.json")
    f = lambda a: np.asarray(a, np.float32)
    for case in g["cases"]:
        y, gamma = orc.adarmsnorm(f(g["x"]), f(case["c"]), f(g["W1"]), f(g["b1"]), f(g["W2"]), f(g["b2"]), g["eps"], return_gate=True)
        assert np.max(np.abs(gamma - np.asarray(case["gamma"]))) <= 1e-7, case["arithmetic"]      # (b1, W2 are exact in fp32; SiLU(1) is not)
        assert np.max(np.abs(y - np.asarray(case["y"]))) <= 1e-6, case["arithmetic"]


def test_eq1_attention_hand_cases_both_oracle_forms():
    g = load("eq1_attention_hand.json")
    d, N = g["d"], g["ring_capacity"]
    f = lambda a: np.asarray(a, np.float32)
    for head0 in (0, 1):                                 # the live token lands in slot head0, the other slot stays dead
        oc = orc.OracleCache(1, 1, 1, d, 1, N, head0=[head0])
        oc.k_ring[:] = g["dead_slot_fill"]; oc.v_ring[:] = g["dead_slot_fill"]
        oc.init_static(0, f(g["k_pinned"]).reshape(1, 1, 1, d), f(g["v_pinned"]).reshape(1, 1, 1, d))
        oc.append_sliding(0, f(g["k_ring_live"]).reshape(1, 1, 1, d), f(g["v_ring_live"]).reshape(1, 1, 1, d))
        for case in g["cases"]:
            for partitioned in (False, True):
                out = oc.attention(0, 0, f(case["q"]).reshape(1, 1, d), f(g["k_dyn"]).reshape(1, 1, d), f(g["v_dyn"]).reshape(1, 1, d),
                                   partitioned=partitioned)
                assert np.max(np.abs(out.reshape(-1) - np.asarray(case["out"]).reshape(-1))) <= 1e-6, (case["arithmetic"], head0, partitioned)


def test_ring_closed_form():
    g = load("ring_closed_form.json")
    N = g["N"]
    oc = orc.OracleCache(1, 1, 1, 4, 1, N, head0=[g["head0"]])
    evicted = 0
    for tick in range(1, 41):
        kv = np.full((1, 1, 1, 4), float(tick), np.float32)
        evicted += oc.append_sliding(0, kv, kv)
        want = g["after_ticks"].get(str(tick))
        if want:
            assert (oc.head[0], oc.count[0], evicted) == (want["head"], want["count"], want["evicted_total"]), tick
    # survivors: ticks 25..40, oldest first, the token of tick t in slot (t - 1) mod 16
    ages = oc.slot_map(0)
    assert [int(oc.k_ring[0, 0, s, 0, 0]) for s in ages[:16]] == list(range(25, 41))
    assert all(s == (t - 1) % 16 for s, t in zip(ages[:16], range(25, 41)))


def test_euler_closed_forms():
    g = load("euler_closed_form.json")
    assert [orc.flow_time(k, 4) for k in range(4)] == g["t_schedule_K4"]
    for case in g["cases"]:
        x = np.asarray(case["x0"], np.float64).copy()
        for k in range(case["K"]):
            v = np.asarray(case["v"], np.float32) if "v" in case else x.astype(np.float32)
            orc.flow_step(x, v, case["K"])
        assert np.max(np.abs(x - np.asarray(case["xK"]))) <= 1e-6, case["arithmetic"]
