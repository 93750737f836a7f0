"""The controller comparison (oracle/controller_study.py): pins of its bookkeeping and cost formula.

Not GPU tests: everything here runs the oracle on small synthetic workloads."""
import numpy as np
import pytest

import oracle
from oracle import controller_study as cs
from paper_2504_00030_b200 import synth


@pytest.fixture(scope="module")
def small():
    return cs.workload(batch=3, vocab=512, steps=90, block=15, seed=77)


def test_fixed_gamma_on_iid_rows_meets_the_geometric_closed_form():
    """All positions alike and independent: with acceptance rate alpha the tokens per step average
    (1 - alpha^(gamma+1)) / (1 - alpha), and the cost per token of Eq. 2 follows from it."""
    batch, vocab, steps, gamma = 16, 512, 400, 5
    cfg = synth.VerifyConfig("iid", batch, 1, 1, 64, vocab, 64, 64, cs.GAMMA_MAX, cs.GAMMA_MAX, cs.GAMMA_MAX, 1.0, 1.0,
                             seed=3)
    cu_q, cu_d = synth.padded_offsets(batch, cs.GAMMA_MAX)
    full = np.full(batch, cs.GAMMA_MAX, np.int32)
    inputs = [synth.make_logits(cfg, full, cu_q, cu_d, step=t, sigma_noise=0.8) for t in range(steps)]
    # alpha of this workload, from the oracle's residual mass on forced rejections (rows are alike)
    li = inputs[0]
    one = np.ones(batch, np.int32)
    res = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept, li.u_sample, 1.0,
                               one, cu_q, cu_d, cs.GAMMA_MAX, force=np.zeros(int(cu_d[-1]), np.int8))
    alpha = float(np.mean(1.0 - res.resid_mass))
    drafted, accepted, issued = cs.run_method("SpecDecode", gamma, cfg, cu_q, cu_d, inputs)
    assert (issued == gamma).all() and (drafted == gamma).all()
    tokens = (accepted + 1).mean()
    closed = (1.0 - alpha ** (gamma + 1)) / (1.0 - alpha)
    sd = np.sqrt((accepted + 1).var() / accepted.size)
    assert abs(tokens - closed) < 5 * sd + 0.02 * closed, (tokens, closed, alpha)
    for c in (4.0, 10.0):
        assert cs.cost_per_token(drafted, accepted, c) == pytest.approx((c + gamma) / tokens, rel=1e-12)


def test_a_threshold_of_zero_changes_nothing(small):
    cfg, cu_q, cu_d, inputs = small
    old = cs.TAU
    try:
        cs.TAU = 0.0
        for plain, plus in (("SpecDecode", "AssistantThreshold"), ("GammaTune", "GammaTune+")):
            a = cs.run_method(plain, 6, cfg, cu_q, cu_d, inputs)
            b = cs.run_method(plus, 6, cfg, cu_q, cu_d, inputs)
            for x, y in zip(a, b):
                np.testing.assert_array_equal(x, y)
    finally:
        cs.TAU = old


def test_bookkeeping_of_every_method(small):
    cfg, cu_q, cu_d, inputs = small
    for m in cs.METHODS:
        drafted, accepted, issued = cs.run_method(m, 8, cfg, cu_q, cu_d, inputs)
        assert (accepted <= drafted).all() and (drafted <= issued).all() and (drafted >= 1).all()
        if m in ("SpecDecode", "AssistantThreshold"):
            assert (issued == 8).all()                       # the cap never moves without Algorithm 1
        else:
            assert issued.min() >= cs.GAMMA_MIN and issued.max() <= cs.GAMMA_MAX and len(np.unique(issued)) > 3
        if m in ("SpecDecode", "GammaTune"):
            assert (drafted == issued).all()                 # no early stop without a threshold
        else:
            assert (drafted < issued).any()


def test_cost_formula_by_hand():
    # two steps, one sequence: 5 drafts with 2 accepted, then 3 drafts all accepted; c = 4:
    # cost (4 + 5) + (4 + 3) = 16 draft units for (2 + 1) + (3 + 1) = 7 tokens
    assert cs.cost_per_token(np.array([[5], [3]]), np.array([[2], [3]]), 4.0) == pytest.approx(16.0 / 7.0)


def test_adaptive_controllers_depend_less_on_the_initial_gamma():
    """The paper's robustness claim (Table 2: spread over gamma_0 of 0.23 for SpecDecode against 0.05 / 0.03),
    on the synthetic regimes: Algorithm 1 forgets gamma_0, a fixed gamma does not."""
    res = cs.study(cs=(7.0,), batch=3, vocab=512, steps=120, block=20, seed=78)[7.0]
    assert res["GammaTune"][1] < 0.3 * res["SpecDecode"][1]
    assert res["GammaTune+"][1] < 0.3 * res["SpecDecode"][1]
    assert res["GammaTune"][0] > 1.0 and res["GammaTune+"][0] > 1.0
