"""The four controllers of the paper's comparison on the device (SpecDecode, AssistantThreshold, GammaTune,
GammaTune+), as modes of the same three calls: every step's drafted length, accepted count, emitted tokens
and next gamma against the oracle's run of oracle/controller_study.py on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
from oracle import controller_study as cs
from paper_2504_00030_b200 import binding as sv
from tests.harness import DEV, AcceptOut, compare_accept, dev, workspace

pytestmark = pytest.mark.gpu


def device_run(method, gamma0, cfg, cu_q, cu_d, inputs, temperature=1.0):
    B, gmax, steps = cfg.batch, cs.GAMMA_MAX, len(inputs)
    adaptive = method in ("GammaTune", "GammaTune+")
    threshold = method in ("AssistantThreshold", "GammaTune+")
    gcfg = sv.GammaConfig(cs.ETA, cs.DELTA, cs.GAMMA_MIN, gmax, sv.SV_GT_PROPOSED if adaptive else sv.SV_GT_FIXED, True)
    d_in = [(dev(li.target_logits), dev(li.draft_logits), dev(li.draft_tokens), dev(li.u_accept), dev(li.u_sample))
            for li in inputs]
    gbar = torch.zeros(B, dtype=torch.float64, device=DEV)
    g = torch.zeros(B, dtype=torch.int32, device=DEV)
    sl = torch.full((B,), 64, dtype=torch.int32, device=DEV)
    d_cq = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    d_cd = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    sv.gamma_tune_init(gbar, g, d_cq, d_cd, gcfg, gamma0)
    n_acc = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = torch.zeros((steps, B, gmax + 1), dtype=torch.int32, device=DEV)
    n_log = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    traj = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    n_dr = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws_s = workspace(sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab))
    ws_d = workspace(sv.spec_draft_stop_workspace_bytes(B, gmax, cfg.vocab))
    for t, (tl, dl, x, ua, us) in enumerate(d_in):           # nothing is read back inside the loop
        gt = g
        if threshold:
            sv.spec_draft_stop(dl, temperature, cs.TAU, g, d_cd, gmax, n_dr[t], ws_d, device_status=status)
            gt = n_dr[t]
        else:
            n_dr[t].copy_(g)
        sv.spec_accept_sample(tl, dl, x, ua, us, temperature, gt, d_cq, d_cd, gmax, n_acc, toks[t], ws_s,
                              device_status=status)
        sv.gamma_tune_update(n_acc, gbar, g, sl, d_cq, d_cd, gcfg, trajectory=traj, accepted_log=n_log, step=t,
                             device_status=status, n_drafted=n_dr[t] if threshold else None)
    torch.cuda.synchronize()
    assert status.item() == 0
    return n_dr.cpu().numpy(), n_log.cpu().numpy(), traj.cpu().numpy(), toks.cpu().numpy()


@pytest.mark.parametrize("method", cs.METHODS)
def test_controller_runs_match_the_oracle(method):
    cfg, cu_q, cu_d, inputs = cs.workload(batch=4, vocab=4096, steps=48, block=8, seed=20250411)
    gamma0 = 6
    drafted, accepted, traj, toks = device_run(method, gamma0, cfg, cu_q, cu_d, inputs)
    o_drafted, o_accepted, o_issued = cs.run_method(method, gamma0, cfg, cu_q, cu_d, inputs)
    # the oracle's own run first: identical unless a near tie sent the two down different paths
    same = np.array_equal(drafted, o_drafted) and np.array_equal(accepted, o_accepted)
    # step by step, following the device through flagged near ties (either decision is legal there)
    threshold = method in ("AssistantThreshold", "GammaTune+")
    mode = oracle.MODE_GT_PROPOSED if method in ("GammaTune", "GammaTune+") else oracle.MODE_FIXED
    gbar, g, _, _ = oracle.gamma_tune_init(cfg.batch, gamma0, cs.GAMMA_MAX, True)
    sl = np.full(cfg.batch, 64, np.int32)
    flagged = 0
    for t, li in enumerate(inputs):
        n_dr = g
        if threshold:
            n_dr, _, flag = oracle.draft_stop(li.draft_logits, 1.0, cs.TAU, g, cu_d)
            assert flag.any() or np.array_equal(drafted[t], n_dr)
            n_dr = drafted[t]
        else:
            np.testing.assert_array_equal(drafted[t], g)
        gpu = AcceptOut(accepted[t], toks[t], None, None, None, 0, 0)
        _, n_pos, n_tok = compare_accept(gpu, li, 1.0, n_dr, cu_q, cu_d, cs.GAMMA_MAX)
        flagged += n_pos + n_tok
        gbar, g, sl, _, _ = oracle.gamma_tune_update(accepted[t], gbar, g, sl, cs.ETA, cs.DELTA, cs.GAMMA_MIN,
                                                     cs.GAMMA_MAX, mode, True, n_drafted=n_dr if threshold else None)
        np.testing.assert_array_equal(traj[t], g)
    assert same or flagged > 0
    # and the cost of Eq. 2 computed from the device's logs is the oracle's
    if same:
        assert cs.cost_per_token(drafted, accepted, 7.0) == cs.cost_per_token(o_drafted, o_accepted, 7.0)
