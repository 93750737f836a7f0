"""Calibration of the target-draft noise sigma for workloads that ask for an acceptance regime.

The vicuna-13B-shaped workload alternates between regimes of acceptance about 0.9 and about 0.3
without saying which noise level gives them.  This script tabulates, with the oracle only, for
noise sigma on a grid:

  * T = 1:  alpha(sigma) = mean over rows of sum_k min(p_k, q_k), the probability that a draft token
            drawn from q is accepted (Section 3 of the paper calls it the acceptance rate).  The
            oracle reports sum_k max(0, p_k - q_k) = 1 - alpha at a rejection, so every position is
            forced to reject and the residual mass is read back;
  * T = 0:  the frequency of argmax(target) == argmax(draft), i.e. of a greedy acceptance.

Inputs are the seeded synthetic logits of the workload (draft ~ N(0, 2^2), target = draft + N(0, sigma^2),
V = 32000).  Run:  python -m oracle.calibrate_sigma [--rows 256]
The chosen values are the C4_SIGMA table of tests/test_gpu_step.py, used by the multi-step tests.
"""
from __future__ import annotations

import argparse

import numpy as np

import oracle
from paper_2504_00030_b200 import synth

GRID = (0.05, 0.1, 0.15, 0.2, 0.25, 0.3, 0.4, 0.5, 0.65, 0.8, 1.0, 1.25, 1.5, 2.0, 2.5, 3.0, 4.0)


def acceptance(sigma: float, rows: int, workload: str = "c4"):
    """(alpha at T = 1, greedy match rate at T = 0) over `rows` seeded row pairs."""
    cfg = synth.scaled(synth.CONFIGS[workload], batch=rows, gamma_lo=1, gamma_hi=1, gamma_max=1)
    gamma = np.ones(rows, np.int32)
    cu_q, cu_d = synth.prefix(gamma)
    li = synth.make_logits(cfg, gamma, cu_q, cu_d, sigma_noise=sigma, temperature=1.0)
    force = np.zeros(rows, np.int8)                                   # reject everywhere: residual mass reported
    res = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept, li.u_sample,
                               1.0, gamma, cu_q, cu_d, 1, force=force)
    alpha = float(np.mean(1.0 - res.resid_mass))
    li0 = synth.make_logits(cfg, gamma, cu_q, cu_d, sigma_noise=sigma, temperature=0.0)
    res0 = oracle.accept_sample(li0.target_logits, li0.draft_logits, li0.draft_tokens, li0.u_accept,
                                li0.u_sample, 0.0, gamma, cu_q, cu_d, 1)
    return alpha, float(np.mean(res0.n_accepted == 1))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=256)
    ap.add_argument("--workload", default="c4")
    args = ap.parse_args()
    oracle.build()
    print(f"workload {args.workload}, {args.rows} row pairs per sigma")
    print("sigma   alpha(T=1)  greedy match(T=0)")
    table = []
    for s in GRID:
        a1, a0 = acceptance(s, args.rows, args.workload)
        table.append((s, a1, a0))
        print(f"{s:5.2f}   {a1:9.4f}  {a0:9.4f}")
    for name, want in (("high", 0.9), ("low", 0.3)):
        s1 = min(table, key=lambda r: abs(r[1] - want))
        s0 = min(table, key=lambda r: abs(r[2] - want))
        print(f"acceptance about {want}: sigma = {s1[0]} at T = 1 (alpha {s1[1]:.3f}), sigma = {s0[0]} at T = 0 "
              f"(match rate {s0[2]:.3f})")


if __name__ == "__main__":
    main()
