"""Pins for the oracle's latency estimator (Eq. 5-6) and its Algorithm 1 loop, against what the paper
prints and against properties that hold for any input; a second, independently written simulation
(plain Python, token lists instead of counters) must agree with it on random streams."""
import os
import random

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "latency_coeffs.txt")


def coeffs():
    out = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            name, a, b, c, d = line.split()
            out[name] = (float(a), float(b), float(c), float(d))
    return out


def test_printed_coefficients_and_intercepts(oracle):
    c = coeffs()
    assert set(c) == {"SLM-1.5B", "LLM-7B", "LLM-14B"}
    # d is the latency of an empty step: the intercepts the appendix prints
    assert oracle.latency_ms(c["SLM-1.5B"], 0, 0) == 27.090929
    assert oracle.latency_ms(c["LLM-7B"], 0, 12345) == 27.040801
    assert oracle.latency_ms(c["LLM-14B"], 0, 0) == 45.118931
    # a decode step is Eq. 5 at N_inf = 1: a * N_kv + (b + c + d)
    for name, (a, b, cc, d) in c.items():
        for n_kv in (0, 1, 1000, 8192, 16384):
            assert oracle.latency_ms(c[name], 1, n_kv) == pytest.approx(a * n_kv + (b + cc + d), rel=1e-15)
    # hand-evaluated values of the printed polynomials
    assert oracle.latency_ms(c["SLM-1.5B"], 1, 0) == pytest.approx(26.970114, abs=1e-12)
    assert oracle.latency_ms(c["LLM-7B"], 512, 4096) == pytest.approx(
        0.000027 * 512 * 4096 + 0.000031 * 512 * 512 - 0.045256 * 512 + 27.040801, rel=1e-15)
    assert oracle.latency_ms(c["LLM-14B"], 100, 2000) == pytest.approx(9.0 + 1.23 - 8.2998 + 45.118931, rel=1e-13)


def test_latency_is_separately_linear_in_each_monomial(oracle):
    # each coefficient multiplies exactly its own monomial (a dropped or swapped term fails here)
    for n_inf, n_kv in [(1, 0), (3, 7), (17, 4000), (544, 8000)]:
        assert oracle.latency_ms((1, 0, 0, 0), n_inf, n_kv) == n_inf * n_kv
        assert oracle.latency_ms((0, 1, 0, 0), n_inf, n_kv) == n_inf * n_inf
        assert oracle.latency_ms((0, 0, 1, 0), n_inf, n_kv) == n_inf
        assert oracle.latency_ms((0, 0, 0, 1), n_inf, n_kv) == 1


def test_alg1_worked_example(oracle):
    # prompt of 5 tokens; the SLM is unsure at its second step, the LLM takes one step and hands back
    r = oracle.alg1_sequence(5, 8, 0.5, 99, [1, 2, 3, 4, 5, 6, 7, 8], [0.1, 0.9] + [0.1] * 6,
                             [11, 12, 13, 14, 15, 16, 17, 18], [0.9, 0.9] + [0.1] * 6,
                             (0, 0, 0, 1), (0, 0, 0, 10))
    assert r["y"].tolist() == [1, 13, 4, 5, 6, 7, 8]        # 2 was discarded, 13 came from the LLM
    assert (r["kept_slm"], r["kept_llm"], r["steps_slm"], r["steps_llm"]) == (6, 1, 7, 1)
    assert r["len"] == 12 and r["L_slm"] == 12 and r["L_llm"] == 7 and r["active"] == 0
    assert r["lat_ms"] == 17.0 and r["done"] == 0 and r["iters"] == 8


def test_alg1_limits(oracle):
    T = 32
    tok = list(range(100, 100 + T))
    one = (0, 0, 0, 1.0)
    # tau above every entropy: the SLM decodes alone, one prefill then decodes
    r = oracle.alg1_sequence(10, T, 5.0, -1, tok, [1.0] * T, tok, [1.0] * T, one, one)
    assert r["y"].tolist() == tok and r["steps_llm"] == 0 and r["L_llm"] == 0 and r["L_slm"] == 10 + T
    # tau below every entropy: the first SLM token is discarded, then the LLM decodes alone
    r = oracle.alg1_sequence(10, T, -1.0, -1, tok, [1.0] * T, tok, [1.0] * T, one, one)
    assert r["steps_slm"] == 1 and r["kept_slm"] == 0 and r["y"].tolist() == tok[1:]
    assert r["L_slm"] == 10 and r["L_llm"] == 10 + T - 1 and r["active"] == 1
    # strictness of the rule: H == tau keeps the SLM token
    r = oracle.alg1_sequence(3, 2, 0.25, -1, [7, 8], [0.25, 0.25], [0, 0], [9.0, 9.0], one, one)
    assert r["y"].tolist() == [7, 8]
    # EOS stops after appending it
    r = oracle.alg1_sequence(3, 10, 5.0, 42, [1, 42, 3] + [0] * 7, [0.0] * 10, [0] * 10, [0.0] * 10, one, one)
    assert r["y"].tolist() == [1, 42] and r["done"] == 1 and r["iters"] == 2
    # T_max = 0
    r = oracle.alg1_sequence(3, 0, 0.5, -1, [], [], [], [], one, one)
    assert r["n_out"] == 0 and r["len"] == 3 and r["lat_ms"] == 0.0


def reference_sim(prompt_len, t_max, tau, eos, ts, es, tl, el, cs, cl):
    """Algorithm 1 again, with explicit caches as Python lists of token positions."""
    seq = ["x"] * prompt_len
    kv = {"SLM": [], "LLM": []}
    active, y, lat = "SLM", [], 0.0
    steps = {"SLM": 0, "LLM": 0}
    for t in range(t_max):
        coef = cs if active == "SLM" else cl
        if len(kv[active]) < len(seq):
            new = seq[len(kv[active]):]
            n_inf, n_kv = len(new), len(kv[active])
            kv[active] = kv[active] + new + ["pending"]
        else:
            n_inf, n_kv = 1, len(kv[active])
            kv[active] = kv[active] + ["pending"]
        lat += coef[0] * n_inf * n_kv + coef[1] * n_inf ** 2 + coef[2] * n_inf + coef[3]
        steps[active] += 1
        H, tok = (es[t], ts[t]) if active == "SLM" else (el[t], tl[t])
        if H > tau:
            if active == "SLM":
                kv["SLM"].pop()
                active = "LLM"
                continue
        elif active == "LLM":
            active = "SLM"
        y.append(tok)
        seq.append(tok)
        if tok == eos:
            break
    return y, len(kv["SLM"]), len(kv["LLM"]), len(seq), lat, steps, active


def test_alg1_against_second_simulation(oracle):
    rng = random.Random(5)
    c = coeffs()
    for trial in range(200):
        T = rng.randint(1, 60)
        P = rng.randint(1, 300)
        tau = rng.choice([0.1, 0.3, 0.5, 1.0])
        ts = [rng.randint(0, 50) for _ in range(T)]
        tl = [rng.randint(0, 50) for _ in range(T)]
        es = [rng.choice([0.0, 0.05, tau, tau + 1e-9, 2.0, 7.0]) for _ in range(T)]
        el = [rng.choice([0.0, 0.05, tau, tau + 1e-9, 2.0, 7.0]) for _ in range(T)]
        eos = rng.choice([-1, 7])
        r = oracle.alg1_sequence(P, T, tau, eos, ts, es, tl, el, c["SLM-1.5B"], c["LLM-7B"])
        y, Ls, Ll, ln, lat, steps, active = reference_sim(P, T, tau, eos, ts, es, tl, el, c["SLM-1.5B"], c["LLM-7B"])
        assert r["y"].tolist() == y and (r["L_slm"], r["L_llm"], r["len"]) == (Ls, Ll, ln)
        assert r["lat_ms"] == pytest.approx(lat, rel=1e-12)
        assert (r["steps_slm"], r["steps_llm"]) == (steps["SLM"], steps["LLM"])
        assert r["active"] == (0 if active == "SLM" else 1)
        # invariants: every kept token is in y; the caches never run ahead of the sequence by more than
        # the one pending entry; the span the next model step would prefill is never negative
        assert r["kept_slm"] + r["kept_llm"] == r["n_out"] == r["len"] - P
        assert r["L_slm"] <= r["len"] and r["L_llm"] <= r["len"]
        assert r["steps_slm"] + r["steps_llm"] == r["iters"]


# ---- Algorithm 1, the R-Stitch+ lines: switch <- (argmax_a pi(a | s_t) = LLM), consulted when H_t > tau ----

def test_alg1_router_switch_worked_example(oracle):
    # prompt of 4 tokens, tau = 0.5.  The SLM is unsure at loop indices 1, 2 and 4; the router keeps the
    # SLM at 1, hands over at 2 (that token is discarded), the LLM stays unsure once and hands back at 4,
    # where the SLM is unsure again and the router keeps it.
    #   t      0     1     2       3          4       5
    #   model  SLM   SLM   SLM->   LLM        LLM->   SLM
    #   H      0.1   0.9   0.9     0.9        0.2     0.9
    #   switch -     0     1       (ignored)  -       0
    ts, es = [1, 2, 3, 4, 5, 6], [0.1, 0.9, 0.9, 0.0, 0.0, 0.9]
    tl, el = [11, 12, 13, 14, 15, 16], [9.0, 9.0, 9.0, 0.9, 0.2, 9.0]
    sw = [1, 0, 1, 0, 1, 0]          # entries at t = 0, 3, 4 must not matter
    r = oracle.alg1_sequence(4, 6, 0.5, 99, ts, es, tl, el, (0, 0, 0, 1), (0, 0, 0, 10), switch_slm=sw)
    assert r["y"].tolist() == [1, 2, 14, 15, 6]
    assert (r["kept_slm"], r["kept_llm"], r["steps_slm"], r["steps_llm"]) == (3, 2, 4, 2)
    # the LLM prefilled x + y = 4 + 2 tokens at t = 3, decoded at t = 4; the SLM prefilled its two missing
    # tokens at t = 5
    assert r["L_llm"] == 8 and r["L_slm"] == 9 and r["len"] == 9 and r["active"] == 0
    assert r["lat_ms"] == 4 * 1.0 + 2 * 10.0
    for flip in (0, 3, 4):           # the router is not consulted there
        s2 = list(sw)
        s2[flip] ^= 1
        r2 = oracle.alg1_sequence(4, 6, 0.5, 99, ts, es, tl, el, (0, 0, 0, 1), (0, 0, 0, 10), switch_slm=s2)
        assert r2["y"].tolist() == r["y"].tolist() and r2["lat_ms"] == r["lat_ms"]


def test_alg1_router_switch_limits(oracle):
    rng = random.Random(11)
    c = coeffs()
    for trial in range(100):
        T, P = rng.randint(1, 50), rng.randint(1, 200)
        tau = rng.choice([0.1, 0.3, 1.0])
        ts = [rng.randint(0, 50) for _ in range(T)]
        tl = [rng.randint(0, 50) for _ in range(T)]
        es = [rng.choice([0.0, tau, tau + 1e-9, 2.0]) for _ in range(T)]
        el = [rng.choice([0.0, tau, tau + 1e-9, 2.0]) for _ in range(T)]
        args = (P, T, tau, -1, ts, es, tl, el, c["SLM-1.5B"], c["LLM-7B"])
        # switch always true is R-Stitch
        plain = oracle.alg1_sequence(*args)
        always = oracle.alg1_sequence(*args, switch_slm=[1] * T)
        assert always["y"].tolist() == plain["y"].tolist() and always["lat_ms"] == plain["lat_ms"]
        assert (always["L_slm"], always["L_llm"], always["active"]) == (plain["L_slm"], plain["L_llm"], plain["active"])
        # switch never true: the SLM decodes alone whatever its entropy (one prefill, then decodes)
        never = oracle.alg1_sequence(*args, switch_slm=[0] * T)
        assert never["y"].tolist() == ts and never["steps_llm"] == 0 and never["kept_llm"] == 0
        assert never["active"] == 0 and never["L_llm"] == 0 and never["L_slm"] == P + T
        # a random router never hands over more often than R-Stitch at the same threshold would let it:
        # every LLM step follows an SLM step with H > tau and switch = 1
        sw = [rng.randint(0, 1) for _ in range(T)]
        mixed = oracle.alg1_sequence(*args, switch_slm=sw)
        handoffs = mixed["steps_slm"] - mixed["kept_slm"]
        assert handoffs <= sum(1 for t in range(T) if es[t] > tau and sw[t])
        assert mixed["kept_slm"] + mixed["kept_llm"] == mixed["n_out"] and mixed["steps_slm"] + mixed["steps_llm"] == mixed["iters"]
