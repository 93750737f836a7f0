"""The paper's comparison of draft-length controllers, replayed with the oracle on synthetic logits.

Section 5 of the paper compares five ways of choosing the speculation length gamma over twelve initial
values gamma_0 (Table 2: mean and spread of the speed-up over plain speculative decoding).  Four of them
are defined by the paper and are run here:

    SpecDecode          gamma fixed at gamma_0                                   (Section 3)
    AssistantThreshold  gamma_0 as the cap, drafting stops when the draft model's top
                        probability falls below tau                              (Section 4.2, without Algorithm 1)
    GammaTune           Algorithm 1 (Eq. 7, Eq. 8) starting from gamma_0         (Section 4.1)
    GammaTune+          Algorithm 1 plus the threshold                            (Section 4.2)

(the fifth, HFHeuristic, is only named by the paper; its rule is not given there).

Every step is taken by the oracle: oracle.draft_stop where a threshold applies, oracle.accept_sample,
oracle.gamma_tune_update.  The cost of a run follows Eq. 2: every step costs one target call (c draft
units, c = T_target / T_draft, Eq. 1; the paper quotes c between 4 and 10) plus one draft call per drafted
token, and yields A + 1 tokens, so

    cost per token = sum_t (c + n_drafted_t) / sum_t (A_t + 1)          [units of T_draft]

For a fixed gamma and independent acceptances this is what Eq. 3-6 evaluate in closed form.

Synthetic workload (model weights and SpecBench are not available): the acceptance regime changes every
`block` steps between easy, moderate and difficult (Section 4, first paragraph) -- the share of hard
positions is 5 %, 30 % and 70 %; a hard position has a flat draft distribution far from the target's, an
easy one a peaked draft distribution that the target nearly shares (paper_2504_00030_b200.synth.mixture_rows).

Run:  python -m oracle.controller_study
"""
from __future__ import annotations

import argparse

import numpy as np

import oracle
from paper_2504_00030_b200 import synth

GAMMA0 = (1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 20, 24)          # the paper's initial values (Section 5)
GAMMA_MAX = 24
HARD_SHARE = (0.05, 0.30, 0.70)                            # easy, moderate, difficult
METHODS = ("SpecDecode", "AssistantThreshold", "GammaTune", "GammaTune+")
ETA, DELTA, GAMMA_MIN, TAU = 0.5, 2.0, 1, 0.02


def workload(batch=4, vocab=4096, steps=240, block=40, seed=20250410):
    """Per-step inputs (full slabs of GAMMA_MAX + 1 rows per sequence), generated once."""
    cfg = synth.VerifyConfig("study", batch, 1, 1, 64, vocab, 64, 64, GAMMA_MAX, GAMMA_MAX, GAMMA_MAX, 1.0, 1.0,
                             seed=seed)
    cu_q, cu_d = synth.padded_offsets(batch, GAMMA_MAX)
    full = np.full(batch, GAMMA_MAX, np.int32)
    inputs = []
    for t in range(steps):
        share = HARD_SHARE[(t // block) % len(HARD_SHARE)]
        rows = synth.mixture_rows(cfg, int(cu_q[-1]), t, share)
        inputs.append(synth.make_logits(cfg, full, cu_q, cu_d, step=t, row_sigmas=rows))
    return cfg, cu_q, cu_d, inputs


def run_method(method, gamma0, cfg, cu_q, cu_d, inputs, temperature=1.0):
    """One run; returns per-step arrays (n_drafted [steps, B], accepted [steps, B], gamma issued [steps, B])."""
    B = cfg.batch
    adaptive = method in ("GammaTune", "GammaTune+")
    threshold = method in ("AssistantThreshold", "GammaTune+")
    mode = oracle.MODE_GT_PROPOSED if adaptive else oracle.MODE_FIXED
    gbar, g, _, _ = oracle.gamma_tune_init(B, gamma0, GAMMA_MAX, True)
    sl = np.full(B, 64, np.int32)
    drafted, accepted, issued = [], [], []
    for li in inputs:
        n_dr = g
        if threshold:
            n_dr, _, _ = oracle.draft_stop(li.draft_logits, temperature, TAU, g, cu_d)
        res = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept, li.u_sample,
                                   temperature, n_dr, cu_q, cu_d, GAMMA_MAX)
        drafted.append(n_dr.copy())
        accepted.append(res.n_accepted.copy())
        issued.append(g.copy())
        gbar, g, sl, _, _ = oracle.gamma_tune_update(res.n_accepted, gbar, g, sl, ETA, DELTA, GAMMA_MIN, GAMMA_MAX,
                                                     mode, True, n_drafted=n_dr if threshold else None)
    return np.array(drafted), np.array(accepted), np.array(issued)


def cost_per_token(drafted, accepted, c):
    """Eq. 2 summed over the steps of a run, per generated token, in units of T_draft."""
    return float((c * drafted.size + drafted.sum()) / (accepted + 1).sum())


def study(cs=(4.0, 7.0, 10.0), **kw):
    """{c: {method: (mean, std) of the speed-up over the mean SpecDecode throughput, over GAMMA0}}"""
    cfg, cu_q, cu_d, inputs = workload(**kw)
    runs = {m: [run_method(m, g0, cfg, cu_q, cu_d, inputs)[:2] for g0 in GAMMA0] for m in METHODS}
    out = {}
    for c in cs:
        thr = {m: np.array([1.0 / cost_per_token(d, a, c) for d, a in runs[m]]) for m in METHODS}
        base = thr["SpecDecode"].mean()
        out[c] = {m: (float(thr[m].mean() / base), float(thr[m].std() / base)) for m in METHODS}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=240)
    ap.add_argument("--batch", type=int, default=4)
    args = ap.parse_args()
    oracle.build()
    res = study(steps=args.steps, batch=args.batch)
    print(f"speed-up over the mean of SpecDecode, mean +- std over gamma_0 in {GAMMA0}")
    print(f"(eta {ETA}, delta {DELTA}, gamma in [{GAMMA_MIN}, {GAMMA_MAX}], tau {TAU}; {args.steps} steps x {args.batch} sequences)")
    print("method              " + "".join(f"c = {c:<14g}" for c in res))
    for m in METHODS:
        print(f"{m:20s}" + "".join(f"{res[c][m][0]:.2f} +- {res[c][m][1]:.2f}      " for c in res))
    print("paper, Table 2 (mean over four model pairs, H100): SpecDecode 1.00 +- 0.23, HFHeuristic 1.11 +- 0.12,")
    print("AssistantThreshold 1.13 +- 0.06, GammaTune 1.15 +- 0.05, GammaTune+ 1.16 +- 0.03")


if __name__ == "__main__":
    main()
