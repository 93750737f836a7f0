"""Pins for the oracle's accept / resample step.

The procedure is an exact sampler (paper Section 3: the output follows the
target distribution), so it is pinned by what the mathematics fixes:
chi-square exactness on small vocabularies, the geometric closed form for the
number of accepted tokens, degenerate cases, a hand example and brute force.
"""
import numpy as np
import pytest
from scipy import stats

import oracle


def logits_of(p, shift=0.0, T=1.0):
    with np.errstate(divide="ignore"):
        return (T * (np.log(np.asarray(p, np.float64)) + shift)).astype(np.float32)


def draw_from(rng, q, n):
    cdf = np.cumsum(q)
    cdf[-1] = 1.0
    return np.minimum((rng.random(n)[:, None] >= cdf[None, :]).sum(1), len(q) - 1).astype(np.int32)


def run_trials(rng, p_rows, q_rows, n_trials, T=1.0):
    """n_trials independent sequences, each with gamma = len(q_rows) positions whose
    target / draft distributions are p_rows[i] / q_rows[i] whatever came before."""
    gamma = len(q_rows)
    V = len(p_rows[0])
    tl = np.tile(np.stack([logits_of(p, T=T) for p in p_rows]), (n_trials, 1))
    dl = np.tile(np.stack([logits_of(q, T=T) for q in q_rows]), (n_trials, 1)) if gamma else \
        np.zeros((0, V), np.float32)
    x = np.stack([draw_from(rng, q, n_trials) for q in q_rows], 1).reshape(-1) if gamma else \
        np.zeros(0, np.int32)
    g = np.full(n_trials, gamma, np.int32)
    cu_q = (np.arange(n_trials + 1) * (gamma + 1)).astype(np.int32)
    cu_d = (np.arange(n_trials + 1) * gamma).astype(np.int32)
    ua = rng.random(n_trials * gamma, dtype=np.float32)
    us = rng.random(n_trials, dtype=np.float32)
    return oracle.accept_sample(tl, dl, x, ua, us, T, g, cu_q, cu_d, gamma), x.reshape(n_trials, gamma)


def chi2_p(samples, probs):
    V = len(probs)
    obs = np.bincount(samples, minlength=V).astype(np.float64)
    keep = np.asarray(probs) > 0
    assert obs[~keep].sum() == 0, "a zero-probability token was emitted"
    exp = np.asarray(probs)[keep] * obs.sum()
    return stats.chisquare(obs[keep], exp).pvalue


@pytest.mark.parametrize("V,gamma,T", [(8, 3, 1.0), (5, 1, 1.0), (17, 4, 0.7), (8, 2, 2.0)])
def test_emitted_tokens_follow_target_distribution(V, gamma, T):
    rng = np.random.default_rng(100 + V + gamma)
    p_rows = [rng.dirichlet(np.ones(V)) for _ in range(gamma + 1)]
    q_rows = [rng.dirichlet(np.ones(V)) for _ in range(gamma)]
    N = 400_000
    res, x = run_trials(rng, p_rows, q_rows, N, T=T)
    n = res.n_accepted
    # token j of the output is emitted whenever n >= j; given that, it must follow p_j
    for j in range(gamma + 1):
        sel = n >= j
        assert sel.sum() > 1000
        pv = chi2_p(res.out_tokens[sel, j], p_rows[j])
        assert pv > 1e-3, (j, pv)
    # accepted prefix is the draft prefix, padding is -1
    for j in range(gamma):
        np.testing.assert_array_equal(res.out_tokens[n > j, j], x[n > j, j])
        assert (res.out_tokens[n < j, j] == -1).all()
    # position 0 acceptance frequency equals sum_k min(p, q)
    alpha0 = np.minimum(p_rows[0], q_rows[0]).sum()
    freq = (n >= 1).mean()
    assert abs(freq - alpha0) < 4 * np.sqrt(alpha0 * (1 - alpha0) / N)


@pytest.mark.parametrize("alpha,gamma,expect", [(0.7, 4, 2.7731), (0.9, 8, 6.1258), (0.3, 8, 1.4285),
                                                (0.5, 1, 1.5)])
def test_expected_tokens_closed_form(alpha, gamma, expect):
    # i.i.d. acceptance rate alpha: E[A + 1] = (1 - alpha^(gamma+1)) / (1 - alpha),
    # P(A = k) = alpha^k (1 - alpha) for k < gamma and alpha^gamma for k = gamma.
    closed = (1 - alpha ** (gamma + 1)) / (1 - alpha)
    assert abs(closed - expect) < 5e-5
    rng = np.random.default_rng(7)
    p = np.array([alpha, 1 - alpha, 0.0])
    q = np.array([alpha, 0.0, 1 - alpha])        # sum min(p, q) = alpha
    N = 300_000
    res, _ = run_trials(rng, [p] * (gamma + 1), [q] * gamma, N)
    tokens = res.n_accepted + 1.0
    assert abs(tokens.mean() - closed) < 4 * tokens.std() / np.sqrt(N)
    pk = np.array([alpha ** k * (1 - alpha) for k in range(gamma)] + [alpha ** gamma])
    assert chi2_p(res.n_accepted, pk) > 1e-3


def test_identical_models_accept_everything():
    rng = np.random.default_rng(11)
    V, gamma, N = 6, 3, 50_000
    rows = [rng.dirichlet(np.ones(V)) for _ in range(gamma + 1)]
    res, x = run_trials(rng, rows, rows[:gamma], N)
    assert (res.n_accepted == gamma).all()
    np.testing.assert_array_equal(res.out_tokens[:, :gamma], x)
    assert chi2_p(res.out_tokens[:, gamma], rows[gamma]) > 1e-3      # bonus token ~ p_gamma
    assert np.nanmax(np.abs(res.ratio - 1.0)) == 0.0


def test_disjoint_supports_reject_at_once():
    rng = np.random.default_rng(12)
    p = np.array([0.5, 0.3, 0.2, 0.0, 0.0])
    q = np.array([0.0, 0.0, 0.0, 0.6, 0.4])
    res, _ = run_trials(rng, [p, p, p], [q, q], 50_000)
    assert (res.n_accepted == 0).all()
    assert chi2_p(res.out_tokens[:, 0], p) > 1e-3                     # residual = p_0
    assert (res.out_tokens[:, 1:] == -1).all()
    np.testing.assert_allclose(res.resid_mass, 1.0, atol=1e-6)


def test_hand_example_two_tokens():
    # p = (3/4, 1/4), q = (1/4, 3/4), x = 1: ratio = (1/4)/(3/4) = 1/3;
    # residual max(0, p - q) = (1/2, 0) -> normalised (1, 0) -> the next token is 0.
    tl = np.stack([logits_of([0.75, 0.25]), logits_of([0.75, 0.25])])
    dl = np.stack([logits_of([0.25, 0.75])])
    common = dict(temperature=1.0, gamma=[1], cu_q=[0, 2], cu_d=[0, 1], gamma_max=1)
    rej = oracle.accept_sample(tl, dl, [1], [0.5], [0.9], **common)
    assert abs(rej.ratio[0] - 1 / 3) < 1e-7
    assert rej.n_accepted[0] == 0 and list(rej.out_tokens[0]) == [0, -1]
    assert abs(rej.resid_mass[0] - 0.5) < 1e-7
    acc = oracle.accept_sample(tl, dl, [1], [0.3], [0.9], **common)
    # accepted: bonus token from p = (3/4, 1/4) with u = 0.9 > 3/4 -> token 1
    assert acc.n_accepted[0] == 1 and list(acc.out_tokens[0]) == [1, 1]
    acc2 = oracle.accept_sample(tl, dl, [1], [0.3], [0.7], **common)
    assert list(acc2.out_tokens[0]) == [1, 0]
    # x = 0: ratio = min(1, (3/4)/(1/4)) = 1 -> accepted for every u in [0, 1)
    one = oracle.accept_sample(tl, dl, [0], [0.99999994], [0.1], **common)
    assert one.ratio[0] == 1.0 and one.n_accepted[0] == 1


def test_log_partition_and_temperature():
    # logits = T * (ln p + c)  =>  softmax(logits / T) = p and ln sum exp(logits / T) = c
    p = np.array([0.5, 0.25, 0.125, 0.125])
    q = np.array([0.125, 0.125, 0.25, 0.5])
    for T in (0.5, 1.0, 3.0):
        tl = np.stack([logits_of(p, 5.0, T), logits_of(p, -2.0, T)])
        dl = np.stack([logits_of(q, 1.5, T)])
        r = oracle.accept_sample(tl, dl, [3], [0.9], [0.3], T, [1], [0, 2], [0, 1], 1)
        assert abs(r.ratio[0] - 0.25) < 1e-6          # p[3]/q[3] = 0.125/0.5
        assert abs(r.logZ_p[0] - 5.0) < 1e-6 and abs(r.logZ_q[0] - 1.5) < 1e-6
        assert r.n_accepted[0] == 0
        # residual (3/8, 1/8, 0, 0)/(1/2): u = 0.3 < 3/4 -> token 0
        assert r.out_tokens[0, 0] == 0 and abs(r.resid_mass[0] - 0.5) < 1e-6


def test_inverse_cdf_is_strict_and_skips_zero_weights():
    # four equal logits: p = 1/4 each, exactly.  smallest k with cum_k > u
    tl = np.zeros((1, 4), np.float32)
    dl = np.zeros((0, 4), np.float32)
    for u, k in [(0.0, 0), (0.2499999, 0), (0.25, 1), (0.5, 2), (0.74, 2), (0.75, 3), (0.99999994, 3)]:
        r = oracle.accept_sample(tl, dl, [], [], [u], 1.0, [0], [0, 1], [0, 0], 0)
        assert r.n_accepted[0] == 0 and r.out_tokens[0, 0] == k, (u, k)
    # zero-weight tokens (logit -inf) can never come out, not even for u = 0
    tl = np.array([[-np.inf, 0.0, -np.inf, 0.0, -np.inf]], np.float32)
    dl = np.zeros((0, 5), np.float32)
    for u, k in [(0.0, 1), (0.49, 1), (0.5, 3), (0.99999994, 3)]:
        r = oracle.accept_sample(tl, dl, [], [], [u], 1.0, [0], [0, 1], [0, 0], 0)
        assert r.out_tokens[0, 0] == k, (u, k)


def test_near_tie_flags():
    tl = np.stack([logits_of([0.75, 0.25]), logits_of([0.75, 0.25])])
    dl = np.stack([logits_of([0.25, 0.75])])
    common = dict(temperature=1.0, gamma=[1], cu_q=[0, 2], cu_d=[0, 1], gamma_max=1)
    u = np.float32(1 / 3)                                   # |u - ratio| ~ 1e-8
    r = oracle.accept_sample(tl, dl, [1], [u], [0.5], **common)
    assert r.accept_flag[0] == 1
    r = oracle.accept_sample(tl, dl, [1], [0.34], [0.5], **common)
    assert r.accept_flag[0] == 0
    # forcing the decision at the flagged position follows the other branch
    acc = oracle.accept_sample(tl, dl, [1], [u], [0.5], force=[1], **common)
    rej = oracle.accept_sample(tl, dl, [1], [u], [0.5], force=[0], **common)
    assert acc.n_accepted[0] == 1 and rej.n_accepted[0] == 0
    # sampled token: u*W on the edge between tokens 0 and 1 of p = (1/4,1/4,1/4,1/4)
    tl4 = np.zeros((1, 4), np.float32)
    r = oracle.accept_sample(tl4, np.zeros((0, 4), np.float32), [], [], [0.25], 1.0, [0], [0, 1],
                             [0, 0], 0)
    assert r.out_tokens[0, 0] == 1 and r.sample_flag[0] == 1 and r.alt_token[0] == 0
    r = oracle.accept_sample(tl4, np.zeros((0, 4), np.float32), [], [], [0.3], 1.0, [0], [0, 1],
                             [0, 0], 0)
    assert r.sample_flag[0] == 0 and r.alt_token[0] == -1


def test_zero_residual_falls_back_to_target():
    # p == q and a forced rejection: max(0, p - q) has no mass, the token comes from p
    p = np.array([0.0, 0.5, 0.5, 0.0])
    tl = np.stack([logits_of(p), logits_of(p)])
    dl = np.stack([logits_of(p)])
    r = oracle.accept_sample(tl, dl, [1], [0.5], [0.6], 1.0, [1], [0, 2], [0, 1], 1, force=[0])
    assert r.n_accepted[0] == 0 and r.out_tokens[0, 0] == 2 and r.resid_mass[0] == 0.0


def test_greedy_brute_force():
    rng = np.random.default_rng(13)
    V, B, gmax = 50, 200, 5
    gamma = rng.integers(0, gmax + 1, B).astype(np.int32)
    cu_q = np.concatenate([[0], np.cumsum(gamma + 1)]).astype(np.int32)
    cu_d = np.concatenate([[0], np.cumsum(gamma)]).astype(np.int32)
    tl = rng.integers(-3, 4, (cu_q[-1], V)).astype(np.float32)       # many ties
    dl = rng.standard_normal((cu_d[-1], V)).astype(np.float32)
    x = np.zeros(cu_d[-1], np.int32)
    for b in range(B):
        for i in range(gamma[b]):
            row = tl[cu_q[b] + i]
            first_max = int(np.flatnonzero(row == row.max())[0])
            x[cu_d[b] + i] = first_max if rng.random() < 0.8 else int(rng.integers(V))
    r = oracle.accept_sample(tl, dl, x, np.zeros(cu_d[-1], np.float32), np.zeros(B, np.float32),
                             0.0, gamma, cu_q, cu_d, gmax)
    for b in range(B):
        n = gamma[b]
        for i in range(gamma[b]):
            row = list(tl[cu_q[b] + i])
            if row.index(max(row)) != x[cu_d[b] + i]:
                n = i
                break
        row = list(tl[cu_q[b] + n])
        want = list(x[cu_d[b]:cu_d[b] + n]) + [row.index(max(row))] + [-1] * (gmax - n)
        assert r.n_accepted[b] == n and list(r.out_tokens[b]) == want


def test_mixed_temperatures_and_ragged_offsets():
    # per-sequence temperature and padded row slabs give the same answers as one-by-one calls
    rng = np.random.default_rng(14)
    V, gmax = 33, 4
    gamma = np.array([4, 0, 2, 3], np.int32)
    T = np.array([1.0, 0.0, 0.7, 0.0], np.float32)
    cu_q = (np.arange(5) * (gmax + 1)).astype(np.int32)
    cu_d = (np.arange(5) * gmax).astype(np.int32)
    tl = rng.standard_normal((cu_q[-1], V)).astype(np.float32)
    dl = (tl.reshape(4, gmax + 1, V)[:, :gmax] + 0.5 * rng.standard_normal((4, gmax, V))).reshape(-1, V).astype(np.float32)
    x = rng.integers(0, V, cu_d[-1]).astype(np.int32)
    ua, us = rng.random(cu_d[-1], dtype=np.float32), rng.random(4, dtype=np.float32)
    full = oracle.accept_sample(tl, dl, x, ua, us, T, gamma, cu_q, cu_d, gmax)
    for b in range(4):
        g = int(gamma[b])
        one = oracle.accept_sample(tl[cu_q[b]:cu_q[b] + g + 1], dl[cu_d[b]:cu_d[b] + g],
                                   x[cu_d[b]:cu_d[b] + g], ua[cu_d[b]:cu_d[b] + g], us[b:b + 1],
                                   T[b], [g], [0, g + 1], [0, g], gmax)
        assert one.n_accepted[0] == full.n_accepted[b]
        np.testing.assert_array_equal(one.out_tokens[0], full.out_tokens[b])


def test_accept_comparison_is_strict():
    # p uniform over 4 tokens (exactly 1/4), q a point mass on token 2 (exactly 1):
    # ratio = 1/4 exactly; u = 1/4 is NOT below it -> reject; the next float32 below is accepted.
    tl = np.zeros((2, 4), np.float32)
    dl = np.array([[-np.inf, -np.inf, 0.0, -np.inf]], np.float32)
    common = dict(temperature=1.0, gamma=[1], cu_q=[0, 2], cu_d=[0, 1], gamma_max=1)
    r = oracle.accept_sample(tl, dl, [2], [0.25], [0.1], **common)
    assert r.ratio[0] == 0.25 and r.n_accepted[0] == 0
    r = oracle.accept_sample(tl, dl, [2], [np.nextafter(np.float32(0.25), np.float32(0))], [0.1], **common)
    assert r.n_accepted[0] == 1
