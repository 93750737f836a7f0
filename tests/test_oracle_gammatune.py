"""Pins for the oracle's GammaTune controller (paper Section 4.1, Algorithm 1)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "gammatune_traces.txt")
MODES = {"P": oracle.MODE_GT_PROPOSED, "L": oracle.MODE_GT_LITERAL}


def load_traces():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = [x.strip() for x in line.split("|")]
        a = [math.inf if t == "inf" else int(t) for t in f[8].split(",")]
        steps = [tuple(s.split(":")) for s in f[9].split()]
        out.append(dict(name=f[0], mode=f[1], eta=float(f[2]), delta=float(f[3]), gmin=int(f[4]),
                        gmax=int(f[5]), g0=int(f[6]), gbar0=float(f[7]), a=a,
                        steps=[(int(A), float(gb), int(g)) for A, gb, g in steps]))
    return out


TRACES = load_traces()


def run_oracle(tr, a_seq, L0=1000):
    gbar = np.array([tr["gbar0"]])
    g = np.array([tr["g0"]], np.int32)
    sl = np.array([L0], np.int32)
    rows = []
    for a in a_seq:
        A = int(min(g[0], a))
        g_old, sl_old = int(g[0]), int(sl[0])
        gbar, g, sl, cq, cd = oracle.gamma_tune_update([A], gbar, g, sl, tr["eta"], tr["delta"],
                                                       tr["gmin"], tr["gmax"], MODES[tr["mode"]])
        assert sl[0] == sl_old - (g_old + 1) + (A + 1) + (g[0] + 1)
        assert list(cq) == [0, g[0] + 1] and list(cd) == [0, g[0]]
        rows.append((A, float(gbar[0]), int(g[0])))
    return rows


@pytest.mark.parametrize("tr", TRACES, ids=[t["name"] for t in TRACES])
def test_hand_traces(tr):
    assert run_oracle(tr, tr["a"]) == tr["steps"]


@pytest.mark.parametrize("tr", TRACES, ids=[t["name"] for t in TRACES])
def test_traces_against_exact_rationals(tr):
    # the same recurrences in exact rational arithmetic; all values are dyadic, so
    # binary64 must reproduce them without any rounding
    eta, delta = Fraction(tr["eta"]), Fraction(tr["delta"])
    gbar, g = Fraction(tr["gbar0"]), tr["g0"]
    for a, (A_want, gbar_want, g_want) in zip(tr["a"], tr["steps"]):
        A = min(g, a)
        fed = A + delta if (A == g and tr["mode"] == "P") else Fraction(A)
        gbar = min(Fraction(tr["gmax"]), max(Fraction(tr["gmin"]), (1 - eta) * gbar + eta * fed))
        g = math.ceil(gbar)
        assert (A, gbar, g) == (A_want, Fraction(gbar_want), g_want)


def test_bounds_and_ceil_invariants():
    rng = np.random.default_rng(0)
    for eta, delta, gmin, gmax in [(0.5, 2.0, 1, 8), (0.3, 1.5, 2, 16), (0.9, 3.0, 1, 12)]:
        B = 64
        gbar, g, cq, cd = oracle.gamma_tune_init(B, 4)
        sl = np.full(B, 500, np.int32)
        for _ in range(200):
            A = np.minimum(g, rng.integers(0, gmax + 2, B)).astype(np.int32)
            gbar, g, sl, cq, cd = oracle.gamma_tune_update(A, gbar, g, sl, eta, delta, gmin, gmax)
            assert (gbar >= gmin).all() and (gbar <= gmax).all()
            assert (g == np.ceil(gbar)).all() and (g >= gmin).all() and (g <= gmax).all()
            assert (np.diff(cq) == g + 1).all() and (np.diff(cd) == g).all()


def test_limits_of_constant_acceptance():
    tr = dict(mode="P", eta=0.5, delta=2.0, gmin=1, gmax=8, g0=2, gbar0=2.0)
    # everything accepted: gamma reaches gamma_max within ceil((gmax-g0)/(eta*delta)) steps and stays
    rows = run_oracle(tr, [math.inf] * 12)
    assert all(r[2] == 8 for r in rows[6:])
    # nothing accepted: gamma decays to gamma_min
    rows = run_oracle(dict(tr, g0=8, gbar0=8.0), [0] * 12)
    assert rows[-1][1:] == (1.0, 1)
    # eta = 0: the fixed-gamma baseline
    rows = run_oracle(dict(tr, eta=0.0, g0=5, gbar0=5.0), [0, 3, math.inf, 1])
    assert [r[2] for r in rows] == [5, 5, 5, 5]
    # literal listing: gamma can never grow
    rows = run_oracle(dict(tr, mode="L", g0=3, gbar0=3.0), [math.inf] * 20)
    assert all(r[2] == 3 for r in rows)


def test_probe_one_past_acceptable_and_binary64_rounding():
    # constant a = 3: gamma settles at a + 1 = 4 while gbar - 3 halves each step; after
    # 52 halvings the gap is below half an ulp of 3, gbar rounds to exactly 3.0, gamma
    # drops to 3, the all-accepted boost fires and gamma returns to 4.
    tr = dict(mode="P", eta=0.5, delta=1.0, gmin=1, gmax=8, g0=8, gbar0=8.0)
    rows = run_oracle(tr, [3] * 80)
    gammas = [r[2] for r in rows]
    assert gammas[:3] == [6, 5, 4]
    first3 = gammas.index(3)
    assert 50 <= first3 <= 56 and rows[first3][1] == 3.0
    assert gammas[first3 + 1] == 4 and rows[first3 + 1][1] == 3.5


def test_fixed_mode_keeps_state():
    gbar, g, sl, cq, cd = oracle.gamma_tune_update([2, 5], [5.0, 5.0], [5, 5], [100, 200], 0.5, 2.0, 1, 8,
                                                   oracle.MODE_FIXED)
    assert list(gbar) == [5.0, 5.0] and list(g) == [5, 5]
    assert list(sl) == [100 - 6 + 3 + 6, 200 - 6 + 6 + 6]


def test_padded_row_offsets():
    gbar, g, sl, cq, cd = oracle.gamma_tune_update([2, 5, 0], [5.0] * 3, [5] * 3, [100] * 3, 0.5, 2.0,
                                                   1, 8, padded_rows=True)
    assert list(cq) == [0, 9, 18, 27] and list(cd) == [0, 8, 16, 24]


def test_cost_model_closed_form():
    # Eq. 6: cost = N / (alpha*gamma + 1) * (c + gamma) * T_draft
    for N, a, g, c in [(100, 0.7, 4, 5), (1000, 0.3, 8, 10), (64, 0.9, 16, 4)]:
        assert abs(oracle.cost_model(N, a, g, c) - N / (a * g + 1) * (c + g)) < 1e-9
