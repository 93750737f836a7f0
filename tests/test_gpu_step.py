"""Whole verify steps: a device-resident multi-step loop (no host read-back between steps)
against the oracle's step-by-step simulation, and the host-buffer entry point."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import (ATTN_ATOL, DEV, AcceptOut, bits_of, compare_accept, dev, dev_bf16, workspace)

pytestmark = pytest.mark.gpu


def run_loop(cfg, steps, gamma0, gcfg, sigmas, L0, append=False, tau=None, n_inputs=None):
    """Runs `steps` verify steps on the device with padded row slabs; every per-step input is
    uploaded before the loop and nothing is read back until it ends.  Returns what the
    oracle needs to replay the same steps, and the device's logs.  With `append` every step
    first writes that step's new keys and values behind the contexts (spec_kv_append).  With `tau`
    the draft stops early (spec_draft_stop): the step runs with n_drafted as its gamma and the
    controller is told both.  Step t draws its noise level from sigmas[t % len(sigmas)].  With
    `n_inputs` only that many distinct input sets are generated per noise level and step t uses set
    t % n_inputs of its level (long runs at full size: the inputs recur, the controller's state does not)."""
    B, gmax = cfg.batch, cfg.gamma_max
    cu_q, cu_d = synth.padded_offsets(B, gmax)
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    seq_len0 = np.full(B, L0, np.int32)
    kv = synth.make_kv(cfg, seq_len0, reserve_tokens=steps * (gmax + 1))
    k, v = dev_bf16(kv.k_pool), dev_bf16(kv.v_pool)
    pool = sv.spec_kv_pool_register(k, v)
    bt = dev(kv.block_table)
    max_len = L0 + steps * (gmax + 1)
    full_gamma = np.full(B, gmax, np.int32)
    made, made_q = {}, {}

    def input_set(t):
        key = (sigmas[t % len(sigmas)], t if n_inputs is None else t % n_inputs)
        if key not in made:
            made[key] = synth.make_logits(cfg, full_gamma, cu_q, cu_d, step=key[1], sigma_noise=key[0])
        return made[key]

    def q_set(t):
        k = t if n_inputs is None else t % n_inputs
        if k not in made_q:
            made_q[k] = synth.make_q(cfg, n_q, step=k)
        return made_q[k]

    inputs = [input_set(t) for t in range(steps)]
    qs = [q_set(t) for t in range(steps)]
    n_kv = n_q * cfg.hkv * cfg.head_dim
    kv_new = [(synth.normal_bf16_bits(cfg.seed, 90, n_kv, 1.0, t).reshape(n_q, cfg.hkv, cfg.head_dim),
               synth.normal_bf16_bits(cfg.seed, 91, n_kv, 1.0, t).reshape(n_q, cfg.hkv, cfg.head_dim))
              for t in range(steps)] if append else []
    d_kv = [(dev_bf16(a), dev_bf16(b)) for a, b in kv_new]
    up, up_q = {}, {}                                   # one device copy per distinct input set
    for li, q in zip(inputs, qs):
        if id(li) not in up:
            up[id(li)] = (dev(li.target_logits), dev(li.draft_logits), dev(li.draft_tokens), dev(li.u_accept),
                          dev(li.u_sample))
        if id(q) not in up_q:
            up_q[id(q)] = dev_bf16(q)
    d_in = [up[id(li)] + (up_q[id(q)],) for li, q in zip(inputs, qs)]

    gbar = torch.zeros(B, dtype=torch.float64, device=DEV)
    g = torch.zeros(B, dtype=torch.int32, device=DEV)
    sl = dev(seq_len0)                                  # KV length including the first block
    d_cq = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    d_cd = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    sv.gamma_tune_init(gbar, g, d_cq, d_cd, gcfg, gamma0)
    n_acc = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = torch.zeros((steps, B, gmax + 1), dtype=torch.int32, device=DEV)
    n_log = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    traj = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    o = torch.zeros((steps, n_q, cfg.hq, cfg.head_dim), dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws_a = workspace(sv.spec_verify_attn_workspace_bytes(B, gmax, cfg.hq, cfg.hkv, cfg.head_dim, max_len))
    ws_s = workspace(sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab))
    ws_d = workspace(sv.spec_draft_stop_workspace_bytes(B, gmax, cfg.vocab))
    n_dr = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    sl0 = sl.clone()
    for t in range(steps):
        tl, dl, x, ua, us, q = d_in[t]
        gt = g                                          # the draft lengths this step runs with
        if tau is not None:
            # the block appended before the step has gamma + 1 positions; the step uses n_drafted + 1 of them
            sv.spec_draft_stop(dl, cfg.temperature, tau, g, d_cd, gmax, n_dr[t], ws_d, device_status=status)
            gt = n_dr[t]
            sl_t = sl - g + gt                          # device arithmetic, no read-back
        else:
            sl_t = sl
        if append:
            sv.spec_kv_append(d_kv[t][0], d_kv[t][1], pool, bt, sl_t, gt, d_cq, gmax, device_status=status)
        sv.spec_verify_attn(q, o[t], pool, bt, sl_t, gt, d_cq, gmax, max_len, ws_a, device_status=status)
        sv.spec_accept_sample(tl, dl, x, ua, us, cfg.temperature, gt, d_cq, d_cd, gmax, n_acc, toks[t], ws_s,
                              device_status=status)
        sv.gamma_tune_update(n_acc, gbar, g, sl_t if tau is not None else sl, d_cq, d_cd, gcfg, trajectory=traj,
                             accepted_log=n_log, step=t, device_status=status,
                             n_drafted=n_dr[t] if tau is not None else None)
        if tau is not None:
            sl = sl_t                                   # updated in place by the controller
    torch.cuda.synchronize()
    assert status.item() == 0
    return dict(kv=kv, inputs=inputs, qs=qs, cu_q=cu_q, cu_d=cu_d, sl0=sl0.cpu().numpy(),
                toks=toks.cpu().numpy(), n_log=n_log.cpu().numpy(), traj=traj.cpu().numpy(),
                o=o, gbar=gbar.cpu().numpy(), sl=sl.cpu().numpy(), kv_new=kv_new,
                k_pool=bits_of(k) if append else None, v_pool=bits_of(v) if append else None,
                n_dr=n_dr.cpu().numpy() if tau is not None else None, tau=tau)


def replay_with_oracle(cfg, run, steps, gamma0, gcfg, check_attn_steps=(), attn_samples=None):
    """The oracle takes the same steps.  At `check_attn_steps` the attention outputs are compared too:
    every row, or with `attn_samples` that many seeded (sequence, row, head) outputs computed one by one."""
    B, gmax = cfg.batch, cfg.gamma_max
    gbar, g, _, _ = oracle.gamma_tune_init(B, gamma0, gmax, True)
    sl = run["sl0"].copy()
    flagged = 0
    scale = float(np.float32(cfg.head_dim ** -0.5))
    kp, vp = run["kv"].k_pool, run["kv"].v_pool
    for t in range(steps):
        li = run["inputs"][t]
        g_issued = g
        if run["tau"] is not None:
            o_n, _, o_flag = oracle.draft_stop(li.draft_logits, cfg.temperature, run["tau"], g, run["cu_d"])
            assert o_flag.any() or np.array_equal(run["n_dr"][t], o_n)
            g = run["n_dr"][t].copy()                   # follow the device through a flagged near tie
            sl = sl - g_issued + g
        if run["kv_new"]:
            kp, vp = oracle.kv_append(run["kv_new"][t][0], run["kv_new"][t][1], kp, vp, run["kv"].strides,
                                      run["kv"].block_table, sl, g, run["cu_q"], cfg.page_size)
        gpu = AcceptOut(run["n_log"][t], run["toks"][t], None, None, None, 0, 0)
        ref, n_pos, n_tok = compare_accept(gpu, li, cfg.temperature, g, run["cu_q"], run["cu_d"], gmax)
        flagged += n_pos + n_tok
        if t in check_attn_steps and attn_samples is not None:
            o_gpu = synth.bf16_to_f32(bits_of(run["o"][t])).astype(np.float64)
            rng = np.random.default_rng(1000 + t)
            for _ in range(attn_samples):
                b = int(rng.integers(B))
                i = int(rng.integers(g[b] + 1))
                h = int(rng.integers(cfg.hq))
                row = run["cu_q"][b] + i
                o_ref, _ = oracle.attn_row(run["qs"][t][row, h], kp, vp, run["kv"].strides, run["kv"].block_table[b],
                                           cfg.page_size, h // cfg.group, int(sl[b]) - (int(g[b]) + 1) + i + 1, scale)
                assert np.abs(o_gpu[row, h] - o_ref).max() <= ATTN_ATOL
        elif t in check_attn_steps:
            o_ref, _ = oracle.verify_attn(run["qs"][t], kp, vp, run["kv"].strides,
                                          run["kv"].block_table, sl, g, run["cu_q"], cfg.hq, cfg.hkv,
                                          cfg.page_size, scale)
            o_gpu = synth.bf16_to_f32(bits_of(run["o"][t])).astype(np.float64)
            for b in range(B):
                rows = slice(run["cu_q"][b], run["cu_q"][b] + g[b] + 1)
                assert np.abs(o_gpu[rows] - o_ref[rows]).max() <= ATTN_ATOL
        # follow the device through near ties (compare_accept has already checked legality)
        gbar, g, sl, _, _ = oracle.gamma_tune_update(run["n_log"][t], gbar, g_issued, sl, gcfg.eta, gcfg.delta,
                                                     gcfg.gamma_min, gcfg.gamma_max, gcfg.mode, True,
                                                     n_drafted=g if run["tau"] is not None else None)
        np.testing.assert_array_equal(run["traj"][t], g)
    np.testing.assert_array_equal(run["gbar"].view(np.int64), gbar.view(np.int64))
    np.testing.assert_array_equal(run["sl"], sl)
    if run["kv_new"]:
        # the caches after the last step: every append, and every overwrite of a rejected position
        np.testing.assert_array_equal(run["k_pool"], kp)
        np.testing.assert_array_equal(run["v_pool"], vp)
    return flagged


@pytest.mark.parametrize("gamma0", [1, 4, 8])
def test_c2_gamma_trajectory_device_resident(gamma0):
    # vicuna-7B shape, gamma in [1, 8] driven by the controller, noise 0.3 / 2.0 / 1.0 in blocks
    cfg = synth.scaled(synth.CONFIGS["c2"], ctx_lo=2048, ctx_hi=2048)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, 8, sv.SV_GT_PROPOSED, True)
    steps = 48
    sig = [0.3] * 16 + [2.0] * 16 + [1.0] * 16
    run = run_loop(cfg, steps, gamma0, gcfg, sig, 2048)
    replay_with_oracle(cfg, run, steps, gamma0, gcfg, check_attn_steps=(0, 17, 47))
    assert run["traj"].min() >= 1 and run["traj"].max() <= 8
    assert len(np.unique(run["traj"])) >= 3            # the controller really moved gamma


@pytest.mark.parametrize("sigma", [0.3, 1.0, 2.0])
@pytest.mark.parametrize("gamma0", [1, 4, 8])
def test_c2_at_its_stated_size(sigma, gamma0):
    """vicuna-7B shape as the workload states it: 512 controller-driven steps from a 2048-token context, one run
    per noise level and initial gamma.  Counts, tokens and trajectories are replayed by the oracle at every
    step, the attention outputs at four of them (the context has grown by then).  The per-step inputs recur
    every 64 steps."""
    cfg = synth.scaled(synth.CONFIGS["c2"], ctx_lo=2048, ctx_hi=2048)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, 8, sv.SV_GT_PROPOSED, True)
    steps = 512
    run = run_loop(cfg, steps, gamma0, gcfg, [sigma], 2048, n_inputs=64)
    replay_with_oracle(cfg, run, steps, gamma0, gcfg, check_attn_steps=(0, 100, 300, 511))
    assert run["traj"].min() >= 1 and run["traj"].max() <= 8
    mean_gamma = run["traj"][64:].mean()
    # more noise, fewer accepted drafts, shorter blocks (the oracle's calibration: alpha 0.88 / 0.62 / 0.32)
    assert {0.3: mean_gamma > 3.0, 1.0: 1.5 < mean_gamma < 3.5, 2.0: mean_gamma < 2.0}[sigma], mean_gamma


# noise levels of the two acceptance regimes, from the oracle's calibration table (oracle/calibrate_sigma.py):
# acceptance about 0.9 / about 0.3 at T = 1 (mean sum min(p, q)) and at T = 0 (greedy match rate)
C4_SIGMA = {1.0: (0.25, 2.0), 0.0: (0.05, 1.0)}


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_c4_alternating_regimes_reduced(T):
    # vicuna-13B shape at reduced batch / heads / context; acceptance regime flips every 8 steps
    cfg = synth.scaled(synth.CONFIGS["c4"], batch=8, hq=4, hkv=4, ctx_lo=600, ctx_hi=600, temperature=T)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, 12, sv.SV_GT_PROPOSED, True)
    steps = 32
    hi, lo = C4_SIGMA[T]
    sig = [hi] * 8 + [lo] * 8
    run = run_loop(cfg, steps, 4, gcfg, sig, 600)
    replay_with_oracle(cfg, run, steps, 4, gcfg, check_attn_steps=(5, 20))
    easy = run["traj"][4:8].mean()
    hard = run["traj"][12:16].mean()
    assert easy > hard                                  # expands when drafts are accepted, contracts otherwise


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_c4_at_its_stated_size(T):
    """vicuna-13B shape as the workload states it: batch 64, 40 heads, 4096-token contexts, gamma in [1, 12]
    driven by the controller for 256 steps, acceptance regimes of about 0.9 and about 0.3 alternating every 64
    steps, greedy and sampling.  Every step's counts, tokens and gammas are replayed by the oracle; attention
    outputs are compared on sampled rows in both regimes.  Eight distinct input sets per regime recur."""
    cfg = synth.scaled(synth.CONFIGS["c4"], temperature=T)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, 12, sv.SV_GT_PROPOSED, True)
    steps = 256
    hi, lo = C4_SIGMA[T]
    sig = [hi] * 64 + [lo] * 64
    run = run_loop(cfg, steps, 4, gcfg, sig, 4096, n_inputs=8)
    replay_with_oracle(cfg, run, steps, 4, gcfg, check_attn_steps=(3, 70, 255), attn_samples=24)
    acc = run["n_log"].astype(np.float64) / np.maximum(np.vstack([np.full((1, cfg.batch), 4), run["traj"][:-1]]), 1)
    easy, hard = run["traj"][32:64].mean(), run["traj"][96:128].mean()
    assert easy > hard + 2.0, (easy, hard)              # long blocks while drafts are accepted, short ones otherwise
    assert acc[32:64].mean() > acc[96:128].mean()


def test_loop_that_appends_each_block_to_the_cache():
    # Llama-8B-like GQA shape, reduced: every step writes its block's keys and values, the controller
    # drops the rejected positions by shortening seq_len, and the next block lands on top of them
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=3, hq=8, hkv=2, ctx_lo=200, ctx_hi=200, vocab=4000)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, cfg.gamma_max, sv.SV_GT_PROPOSED, True)
    steps = 20
    sig = [0.3] * 5 + [2.5] * 5
    run = run_loop(cfg, steps, 4, gcfg, sig, 200, append=True)
    replay_with_oracle(cfg, run, steps, 4, gcfg, check_attn_steps=(0, 7, 19))
    assert (run["n_log"] < run["traj"].max()).any()     # there were rejections to roll back
    assert (run["k_pool"] != run["kv"].k_pool).any()


def test_loop_with_early_stop_and_cache_append():
    # GammaTune+ over many steps: the draft stops at the first low-confidence position, the shortened block
    # is appended, verified and accepted, and the controller keeps comparing with the gamma it issued
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=4, hq=8, hkv=2, ctx_lo=150, ctx_hi=150, vocab=3000)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, cfg.gamma_max, sv.SV_GT_PROPOSED, True)
    steps = 16
    # a threshold that about one draft position in seven falls below
    cu_q, cu_d = synth.padded_offsets(cfg.batch, cfg.gamma_max)
    full = np.full(cfg.batch, cfg.gamma_max, np.int32)
    li0 = synth.make_logits(cfg, full, cu_q, cu_d, step=0, sigma_noise=0.4)
    _, top, _ = oracle.draft_stop(li0.draft_logits, cfg.temperature, 0.0, full, cu_d)
    tau = float(np.quantile(top, 0.15))
    run = run_loop(cfg, steps, 6, gcfg, [0.4] * 4 + [2.0] * 4, 150, append=True, tau=tau)
    replay_with_oracle(cfg, run, steps, 6, gcfg, check_attn_steps=(0, 9, 15))
    issued = np.vstack([np.full((1, cfg.batch), 6), run["traj"][:-1]])
    assert (run["n_dr"] < issued).any() and (run["n_dr"] == issued).any()     # some drafts stopped early, some did not


def test_step_from_host_buffers_matches_device_calls():
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=4, ctx_lo=300, ctx_hi=900, vocab=32000)
    B, gmax = cfg.batch, cfg.gamma_max
    seq_len, gamma = synth.draw_lengths(cfg)
    cu_q, cu_d = synth.prefix(gamma)
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    kv = synth.make_kv(cfg, seq_len, reserve_tokens=gmax + 1)
    li = synth.make_logits(cfg, gamma, cu_q, cu_d)
    q = synth.make_q(cfg, n_q)
    k, v = dev_bf16(kv.k_pool), dev_bf16(kv.v_pool)
    pool = sv.spec_kv_pool_register(k, v)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, gmax, sv.SV_GT_PROPOSED)
    max_len = int(seq_len.max()) + gmax + 1
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    q_h = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).pin_memory()
    hosts = dict(tl=pin(li.target_logits), dl=pin(li.draft_logits), x=pin(li.draft_tokens),
                 ua=pin(li.u_accept), us=pin(li.u_sample))
    out_h = dict(n=torch.zeros(B, dtype=torch.int32).pin_memory(),
                 tok=torch.zeros((B, gmax + 1), dtype=torch.int32).pin_memory(),
                 g=torch.zeros(B, dtype=torch.int32).pin_memory(),
                 o=torch.zeros((n_q, cfg.hq, cfg.head_dim), dtype=torch.bfloat16).pin_memory())
    # device staging + state
    d = dict(q=torch.zeros((n_q, cfg.hq, cfg.head_dim), dtype=torch.bfloat16, device=DEV),
             o=torch.zeros((n_q, cfg.hq, cfg.head_dim), dtype=torch.bfloat16, device=DEV),
             tl=torch.zeros((n_q, cfg.vocab), dtype=torch.float32, device=DEV),
             dl=torch.zeros((n_d, cfg.vocab), dtype=torch.float32, device=DEV),
             x=torch.zeros(n_d, dtype=torch.int32, device=DEV),
             ua=torch.zeros(n_d, dtype=torch.float32, device=DEV),
             us=torch.zeros(B, dtype=torch.float32, device=DEV),
             n=torch.zeros(B, dtype=torch.int32, device=DEV),
             tok=torch.zeros((B, gmax + 1), dtype=torch.int32, device=DEV))
    gbar = dev(gamma.astype(np.float64))
    g, sl, cq, cd = dev(gamma), dev(seq_len), dev(cu_q), dev(cu_d)
    ws_a = workspace(sv.spec_verify_attn_workspace_bytes(B, gmax, cfg.hq, cfg.hkv, cfg.head_dim, max_len))
    ws_s = workspace(sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab))
    io = sv.step_host_io(q_h, hosts["tl"], hosts["dl"], hosts["x"], hosts["ua"], hosts["us"], n_q, n_d,
                         out_h["n"], out_h["tok"], out_h["g"], out_h["o"])
    ap = sv.attn_params(d["q"], d["o"], pool, dev(kv.block_table), sl, g, cq, gmax, max_len)
    sp = sv.accept_params(d["tl"], d["dl"], d["x"], d["ua"], d["us"], cfg.temperature, g, cq, cd, gmax,
                          d["n"], d["tok"])
    gp = sv.gamma_params(d["n"], gbar, g, sl, cq, cd, gcfg)
    sv.spec_verify_step_host(io, ap, ws_a, sp, ws_s, gp)
    torch.cuda.synchronize()
    # oracle on the same host arrays
    gpu = AcceptOut(out_h["n"].numpy(), out_h["tok"].numpy(), None, None, None, 0, 0)
    ref, _, _ = compare_accept(gpu, li, cfg.temperature, gamma, cu_q, cu_d, gmax)
    _, g_next, sl_next, _, _ = oracle.gamma_tune_update(out_h["n"].numpy(), gamma.astype(np.float64), gamma,
                                                        seq_len, 0.5, 2.0, 1, gmax)
    np.testing.assert_array_equal(out_h["g"].numpy(), g_next)
    np.testing.assert_array_equal(sl.cpu().numpy(), sl_next)
    o_ref, _ = oracle.verify_attn(q, kv.k_pool, kv.v_pool, kv.strides, kv.block_table, seq_len, gamma, cu_q,
                                  cfg.hq, cfg.hkv, cfg.page_size, float(np.float32(cfg.head_dim ** -0.5)))
    o_gpu = synth.bf16_to_f32(bits_of(out_h["o"])).astype(np.float64)
    assert np.abs(o_gpu - o_ref).max() <= ATTN_ATOL
