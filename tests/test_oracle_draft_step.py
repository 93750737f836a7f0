"""Pins of the oracle's drafting step with the confidence stop (paper Section 4.2): the token drawn from
the draft distribution, its top probability, and the bookkeeping of a drafting loop.  CPU only."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle


def state(B, n_rows):
    return (np.zeros(B, np.int32), np.ones(B, np.int32), np.full(n_rows, -1, np.int32),
            np.full(n_rows, np.nan, np.float64))


def one_step(d, T, tau, u, gamma, cu_d, st):
    n, act, tok, top = st
    return oracle.draft_step(np.asarray(d, np.float32), T, tau, np.asarray(u, np.float32), gamma, cu_d, n, act, tok,
                             top)


def test_uniform_row_is_floor_of_u_times_v():
    # equal logits: q_k = 1/V, smallest k with (k+1)/V > u
    V = 40
    for u in (0.0, 0.013, 0.5, 0.74, 0.999):
        st = state(1, 1)
        one_step(np.zeros((1, V)), 1.0, 0.0, [u], [1], [0, 1], st)
        assert st[2][0] == int(np.floor(np.float32(u) * V))
        assert st[3][0] == pytest.approx(1.0 / V, rel=1e-12)


def test_two_token_closed_form_and_temperature():
    # logits (ln 3, 0): q = (3/4, 1/4) at T = 1; (sqrt 3, 1) / (sqrt 3 + 1) at T = 2
    d = np.array([[np.log(3.0), 0.0]])
    for T, q0 in ((1.0, 0.75), (2.0, np.sqrt(3.0) / (np.sqrt(3.0) + 1.0))):
        for u in (q0 - 1e-3, q0 + 1e-3):
            st = state(1, 1)
            one_step(d, T, 0.0, [u], [1], [0, 1], st)
            assert st[2][0] == (0 if u < q0 else 1)
            assert st[3][0] == pytest.approx(q0, abs=1e-7)


def test_zero_probability_tokens_are_never_drawn():
    d = np.array([[-np.inf, 0.0, -np.inf, 0.0, -np.inf]], np.float32)
    for u, want in ((0.0, 1), (0.49, 1), (0.51, 3), (0.99999, 3)):
        st = state(1, 1)
        one_step(d, 1.0, 0.0, [u], [1], [0, 1], st)
        assert st[2][0] == want


def test_against_numpy_cumsum_searchsorted():
    r = np.random.default_rng(5)
    B, V = 7, 513
    d = (r.standard_normal((B, V)) * 2.0).astype(np.float32)
    T = np.array([0.5, 0.7, 1.0, 1.0, 1.3, 2.0, 4.0], np.float32)
    u = r.random(B).astype(np.float32)
    gamma = np.full(B, 3, np.int32)
    cu_d = np.arange(B + 1, dtype=np.int32) * 3
    st = state(B, 3 * B)
    one_step(d, T, 0.0, u, gamma, cu_d, st)
    for b in range(B):
        q = softmax(d[b].astype(np.float64) / np.float64(T[b]))
        cdf = np.cumsum(q)
        want = int(np.searchsorted(cdf, np.float64(u[b]) * cdf[-1], side="right"))
        assert st[2][cu_d[b]] == want
        assert st[3][cu_d[b]] == pytest.approx(q.max(), rel=1e-12)
    assert (st[0] == 1).all()


def test_frequencies_follow_the_distribution():
    # 4000 draws from one 6-token row: chi-square against q (5 degrees of freedom, 0.999 quantile 20.5)
    r = np.random.default_rng(11)
    V, N = 6, 4000
    row = np.array([0.3, -1.0, 1.2, 0.0, -0.4, 0.8], np.float32)
    d = np.tile(row, (N, 1))
    u = r.random(N).astype(np.float32)
    st = state(N, N)
    one_step(d, 1.0, 0.0, u, np.ones(N, np.int32), np.arange(N + 1, dtype=np.int32), st)
    q = softmax(row.astype(np.float64))
    counts = np.bincount(st[2], minlength=V)
    assert ((counts - N * q) ** 2 / (N * q)).sum() < 20.5


def test_invariant_under_a_shift_of_the_logits():
    r = np.random.default_rng(2)
    d = r.standard_normal((5, 300)).astype(np.float32)
    u = r.random(5).astype(np.float32)
    a, b = state(5, 5), state(5, 5)
    g, cd = np.ones(5, np.int32), np.arange(6, dtype=np.int32)
    one_step(d, 0.9, 0.0, u, g, cd, a)
    one_step(d + np.float32(8.0), 0.9, 0.0, u, g, cd, b)     # the shift rounds the logits by 1e-6: tokens only
    assert (a[2] == b[2]).all()


def test_greedy_takes_the_lowest_argmax_and_never_stops_early():
    d = np.array([[0.0, 2.0, 2.0, 1.0], [5.0, 1.0, 0.0, 5.0]], np.float32)
    st = state(2, 4)
    g, cd = np.array([2, 2], np.int32), np.array([0, 2, 4], np.int32)
    one_step(d, 0.0, 0.99, [0.7, 0.7], g, cd, st)
    assert list(st[2]) == [1, -1, 0, -1]
    assert st[3][0] == 1.0 and st[3][2] == 1.0
    assert list(st[1]) == [1, 1] and list(st[0]) == [1, 1]
    one_step(d, 0.0, 0.99, [0.1, 0.1], g, cd, st)
    assert list(st[2]) == [1, 1, 0, 0]
    assert list(st[1]) == [0, 0] and list(st[0]) == [2, 2]       # the cap gamma ends the drafting


def test_loop_reproduces_the_block_form_of_the_stop():
    """A drafting loop of steps ends with the n_drafted and top probabilities that oracle.draft_stop gives for
    the same rows taken as a block (the low-confidence token is the last one kept)."""
    r = np.random.default_rng(8)
    B, V, gmax, tau = 6, 64, 5, 0.35
    gamma = np.array([5, 3, 0, 5, 1, 4], np.int32)
    cu_d = np.zeros(B + 1, np.int32)
    cu_d[1:] = np.cumsum(gamma)
    n_rows = int(cu_d[-1])
    sig = r.choice([0.5, 3.0], size=n_rows)
    block = (r.standard_normal((n_rows, V)) * sig[:, None]).astype(np.float32)
    st = state(B, max(n_rows, 1))
    st[1][:] = gamma > 0
    for i in range(gmax):
        d = np.zeros((B, V), np.float32)
        for b in range(B):
            if i < gamma[b]:
                d[b] = block[cu_d[b] + i]
        one_step(d, 1.0, tau, r.random(B).astype(np.float32), gamma, cu_d, st)
    n_ref, top_ref, _ = oracle.draft_stop(block, 1.0, tau, gamma, cu_d)
    assert (st[0] == n_ref).all()
    assert (st[1] == 0).all()
    for b in range(B):
        for i in range(int(n_ref[b])):
            assert st[3][cu_d[b] + i] == pytest.approx(top_ref[cu_d[b] + i], rel=1e-12)
            assert st[2][cu_d[b] + i] >= 0
        for i in range(int(n_ref[b]), int(gamma[b])):
            assert st[2][cu_d[b] + i] == -1                       # never drafted


def test_inactive_sequences_are_left_alone_and_flags_are_raised():
    d = np.zeros((2, 4), np.float32)              # q = 1/4 each, exactly
    st = state(2, 2)
    st[1][0] = 0
    alt, sflag, cflag = one_step(d, 1.0, 0.25, [0.5, 0.5], np.array([1, 1], np.int32),
                                 np.array([0, 1, 2], np.int32), st)
    assert st[2][0] == -1 and st[0][0] == 0 and np.isnan(st[3][0])
    assert cflag[1] == 1                    # top probability 1/4 against tau = 1/4
    assert st[2][1] == 2 and sflag[1] == 1 and alt[1] == 1       # u = 1/2 sits on the CDF edge between 1 and 2


def test_confidence_equal_to_the_threshold_keeps_drafting():
    # q = 1/4 each and tau = 1/4: the stop needs c < tau (as in the block form), so the sequence stays active
    st = state(1, 2)
    one_step(np.zeros((1, 4), np.float32), 1.0, 0.25, [0.1], np.array([2], np.int32), np.array([0, 2], np.int32), st)
    assert st[1][0] == 1 and st[0][0] == 1
    n_block, _, _ = oracle.draft_stop(np.zeros((2, 4), np.float32), 1.0, 0.25, [2], [0, 2])
    assert n_block[0] == 2
