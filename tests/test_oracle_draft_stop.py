"""Pins of the oracle's GammaTune+ early stop (paper Section 4.2) and of the controller's
bookkeeping when the draft stopped early.  CPU only."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle


def rows(*vals):
    return np.array(vals, np.float32)


def test_two_token_closed_forms():
    # logits (ln 3, 0): top probability 3/4 at T = 1 and sqrt(3) / (sqrt(3) + 1) at T = 2
    d = rows([np.log(3.0), 0.0])
    _, top, _ = oracle.draft_stop(d, 1.0, 0.5, [1], [0, 1])
    assert top[0] == pytest.approx(0.75, abs=1e-7)
    _, top, _ = oracle.draft_stop(d, 2.0, 0.5, [1], [0, 1])
    assert top[0] == pytest.approx(np.sqrt(3.0) / (np.sqrt(3.0) + 1.0), abs=1e-7)


def test_uniform_and_peaked_rows():
    V = 37
    d = np.zeros((2, V), np.float32)
    d[1, 5] = 60.0
    _, top, _ = oracle.draft_stop(d, 1.0, 0.5, [2], [0, 2])
    assert top[0] == pytest.approx(1.0 / V, rel=1e-12)       # nothing to choose between
    assert top[1] == pytest.approx(1.0, abs=1e-12)


def logits_with_confidence(conf, V=8):
    """Rows whose top probability at T = 1 is exactly conf[i]: one token at ln(c (V-1) / (1-c)), the rest at 0."""
    d = np.zeros((len(conf), V), np.float64)
    for i, c in enumerate(conf):
        d[i, (3 * i) % V] = np.log(c * (V - 1) / (1.0 - c))
    return d.astype(np.float32)


@pytest.mark.parametrize("tau,expect", [(0.5, 3), (0.95, 1), (0.1, 4), (0.85, 2), (0.0, 4)])
def test_stop_rule_on_a_confidence_sequence(tau, expect):
    # confidences 0.9, 0.8, 0.4, 0.9: the first position below tau is the last one drafted
    d = logits_with_confidence([0.9, 0.8, 0.4, 0.9])
    n, top, _ = oracle.draft_stop(d, 1.0, tau, [4], [0, 4])
    np.testing.assert_allclose(top, [0.9, 0.8, 0.4, 0.9], atol=1e-6)
    assert n[0] == expect


def test_never_more_than_gamma_and_gamma_zero():
    d = logits_with_confidence([0.2, 0.2, 0.2])
    n, _, _ = oracle.draft_stop(d, 1.0, 0.5, [3, 0], [0, 3, 3])
    assert n.tolist() == [1, 0]
    d = logits_with_confidence([0.9, 0.9, 0.2])            # the last position is the low one: all three kept
    n, _, _ = oracle.draft_stop(d, 1.0, 0.5, [3], [0, 3])
    assert n.tolist() == [3]


def test_greedy_draft_never_stops():
    d = logits_with_confidence([0.2, 0.2, 0.2])
    n, top, _ = oracle.draft_stop(d, 0.0, 1.0, [3], [0, 3])
    assert n.tolist() == [3] and (top == 1.0).all()


def test_against_scipy_softmax_ragged_batch():
    rng = np.random.default_rng(3)
    gamma = np.array([3, 0, 5, 1], np.int32)
    cu_d = np.concatenate([[0], np.cumsum(gamma)]).astype(np.int32)
    d = (rng.standard_normal((int(cu_d[-1]), 301)) * 3.0).astype(np.float32)
    T = np.array([1.0, 0.7, 0.3, 2.0], np.float32)
    tau = 0.12
    n, top, _ = oracle.draft_stop(d, T, tau, gamma, cu_d)
    for b in range(4):
        conf = [softmax(d[r].astype(np.float64) / float(T[b])).max() for r in range(cu_d[b], cu_d[b + 1])]
        np.testing.assert_allclose(top[cu_d[b]:cu_d[b + 1]], conf, rtol=1e-12)
        below = [i for i, c in enumerate(conf) if c < tau]
        assert n[b] == (min(gamma[b], below[0] + 1) if below else gamma[b])


def test_monotone_in_threshold_and_temperature():
    rng = np.random.default_rng(4)
    d = (rng.standard_normal((6, 64)) * 2.0).astype(np.float32)
    last = 7
    for tau in (0.0, 0.05, 0.1, 0.2, 0.4, 0.8, 1.0):
        n, _, _ = oracle.draft_stop(d, 1.0, tau, [6], [0, 6])
        assert n[0] <= last
        last = n[0]
    _, cold, _ = oracle.draft_stop(d, 0.5, 0.5, [6], [0, 6])
    _, hot, _ = oracle.draft_stop(d, 2.0, 0.5, [6], [0, 6])
    assert (cold > hot).all()                              # a lower temperature sharpens every row


def test_near_threshold_is_flagged():
    d = logits_with_confidence([0.5, 0.9])
    _, top, flag = oracle.draft_stop(d, 1.0, float(top_of(d)), [2], [0, 2])
    assert flag.tolist() == [1, 0]


def top_of(d):
    return softmax(d[0].astype(np.float64)).max()


def test_controller_bookkeeping_after_an_early_stop():
    # gamma 4 issued, the draft stopped after 2, both accepted: no expansion (A != gamma), and the
    # cache held 2 + 1 new positions, of which A + 1 stay
    gbar, g, sl, cq, cd = oracle.gamma_tune_update([2], [4.0], [4], [100], 0.5, 2.0, 1, 8, n_drafted=[2])
    assert gbar[0] == 3.0 and g[0] == 3                    # 0.5 * 4 + 0.5 * 2
    assert sl[0] == 100 - 3 + 3 + 4
    # without an early stop the same call accounts for gamma + 1 appended positions
    _, _, sl2, _, _ = oracle.gamma_tune_update([2], [4.0], [4], [100], 0.5, 2.0, 1, 8)
    assert sl2[0] == 100 - 5 + 3 + 4
    # n_drafted == gamma is the plain update, expansion included
    a = oracle.gamma_tune_update([4], [4.0], [4], [100], 0.5, 2.0, 1, 8, n_drafted=[4])
    b = oracle.gamma_tune_update([4], [4.0], [4], [100], 0.5, 2.0, 1, 8)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    assert a[0][0] == 5.0                                   # 0.5 * 4 + 0.5 * (4 + 2)
