"""gamma_tune_update on the GPU against the oracle: bit-exact gamma_bar, gamma, seq_len, offsets."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from tests.harness import DEV, dev
from tests.test_oracle_gammatune import MODES, TRACES

pytestmark = pytest.mark.gpu


def gpu_state(B, g0, gbar0, L0):
    return (torch.full((B,), float(gbar0), dtype=torch.float64, device=DEV),
            torch.full((B,), int(g0), dtype=torch.int32, device=DEV),
            torch.full((B,), int(L0), dtype=torch.int32, device=DEV),
            torch.zeros(B + 1, dtype=torch.int32, device=DEV),
            torch.zeros(B + 1, dtype=torch.int32, device=DEV))


@pytest.mark.parametrize("tr", TRACES, ids=[t["name"] for t in TRACES])
def test_hand_traces_on_device(tr):
    cfg = sv.GammaConfig(tr["eta"], tr["delta"], tr["gmin"], tr["gmax"], MODES[tr["mode"]])
    gbar, g, sl, cq, cd = gpu_state(1, tr["g0"], tr["gbar0"], 1000)
    for a, (A_want, gbar_want, g_want) in zip(tr["a"], tr["steps"]):
        A = int(min(int(g.item()), a))
        assert A == A_want
        sv.gamma_tune_update(dev(np.array([A], np.int32)), gbar, g, sl, cq, cd, cfg)
        assert gbar.item() == gbar_want and g.item() == g_want
        assert cq.tolist() == [0, g_want + 1] and cd.tolist() == [0, g_want]


@pytest.mark.parametrize("B,padded", [(1, False), (7, False), (300, False), (1000, True), (64, True)])
@pytest.mark.parametrize("eta,delta,gmin,gmax,mode", [(0.5, 2.0, 1, 8, 1), (0.3, 1.7, 2, 16, 1),
                                                      (0.9, 0.5, 0, 12, 2), (0.5, 2.0, 1, 8, 0)])
def test_random_trajectories_bit_exact(B, padded, eta, delta, gmin, gmax, mode):
    rng = np.random.default_rng(B * 31 + gmax)
    cfg = sv.GammaConfig(eta, delta, gmin, gmax, mode, padded)
    g0 = min(4, gmax)
    gbar, g, sl, cq, cd = gpu_state(B, g0, g0, 5000)
    sv.gamma_tune_init(gbar, g, cq, cd, cfg, g0)
    o_gbar, o_g, o_cq, o_cd = oracle.gamma_tune_init(B, g0, gmax, padded)
    o_sl = np.full(B, 5000, np.int32)
    np.testing.assert_array_equal(cq.cpu().numpy(), o_cq)
    steps = 60
    traj = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    alog = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    want_traj = np.zeros((steps, B), np.int32)
    for t in range(steps):
        A = np.minimum(o_g, rng.integers(0, gmax + 2, B)).astype(np.int32)
        sv.gamma_tune_update(dev(A), gbar, g, sl, cq, cd, cfg, trajectory=traj, accepted_log=alog, step=t)
        o_gbar, o_g, o_sl, o_cq, o_cd = oracle.gamma_tune_update(A, o_gbar, o_g, o_sl, eta, delta, gmin,
                                                                 gmax, mode, padded)
        want_traj[t] = o_g
        # bit-exact: compare the float64 bit patterns
        np.testing.assert_array_equal(gbar.cpu().numpy().view(np.int64), o_gbar.view(np.int64))
        np.testing.assert_array_equal(g.cpu().numpy(), o_g)
        np.testing.assert_array_equal(sl.cpu().numpy(), o_sl)
        np.testing.assert_array_equal(cq.cpu().numpy(), o_cq)
        np.testing.assert_array_equal(cd.cpu().numpy(), o_cd)
    np.testing.assert_array_equal(traj.cpu().numpy(), want_traj)


def test_long_run_rounding_event_matches():
    # constant a = 3 with eta = 1/2: after ~52 halvings gamma_bar rounds to exactly 3.0
    cfg = sv.GammaConfig(0.5, 1.0, 1, 8, sv.SV_GT_PROPOSED)
    gbar, g, sl, cq, cd = gpu_state(1, 8, 8.0, 100000)
    o = (np.array([8.0]), np.array([8], np.int32), np.array([100000], np.int32))
    for t in range(512):
        A = np.array([min(int(o[1][0]), 3)], np.int32)
        sv.gamma_tune_update(dev(A), gbar, g, sl, cq, cd, cfg)
        o = oracle.gamma_tune_update(A, *o, 0.5, 1.0, 1, 8)[:3]
        assert gbar.item() == o[0][0] and g.item() == o[1][0] and sl.item() == o[2][0]


def test_checkpoint_resume():
    cfg = sv.GammaConfig(0.25, 2.0, 1, 12, sv.SV_GT_PROPOSED)
    rng = np.random.default_rng(3)
    B = 32
    A_seq = [rng.integers(0, 13, B).astype(np.int32) for _ in range(20)]

    def run(state, lo, hi):
        for t in range(lo, hi):
            A = torch.minimum(dev(A_seq[t]), state[1])
            sv.gamma_tune_update(A, *state, cfg)
        return state
    full = run(gpu_state(B, 2, 2.0, 900), 0, 20)
    half = run(gpu_state(B, 2, 2.0, 900), 0, 10)
    saved = [t.cpu().clone() for t in half]                  # checkpoint: plain copies of the state
    resumed = run(tuple(t.to(DEV) for t in saved), 10, 20)
    for a, b in zip(full, resumed):
        assert torch.equal(a, b)


def test_out_of_range_gamma_sets_status_and_clamps():
    cfg = sv.GammaConfig(0.5, 2.0, 1, 8, sv.SV_GT_PROPOSED)
    gbar, g, sl, cq, cd = gpu_state(2, 4, 4.0, 100)
    g[1] = 99
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sv.gamma_tune_update(dev(np.array([1, 1], np.int32)), gbar, g, sl, cq, cd, cfg, device_status=status)
    assert status.item() & sv.SV_DEV_BAD_GAMMA
    assert 1 <= g[1].item() <= 8


def test_host_errors():
    cfg = sv.GammaConfig(1.5, 2.0, 1, 8, sv.SV_GT_PROPOSED)
    gbar, g, sl, cq, cd = gpu_state(2, 4, 4.0, 100)
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.gamma_tune_update(dev(np.array([1, 1], np.int32)), gbar, g, sl, cq, cd, cfg)
    assert e.value.status == sv.SV_EINVAL
