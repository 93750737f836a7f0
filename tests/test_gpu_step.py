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


def run_loop(cfg, steps, gamma0, gcfg, sigmas, L0):
    """Runs `steps` verify steps on the device with padded row slabs; every per-step input is
    uploaded before the loop and nothing is read back until it ends.  Returns what the
    oracle needs to replay the same steps, and the device's logs."""
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
    inputs = [synth.make_logits(cfg, full_gamma, cu_q, cu_d, step=t, sigma_noise=sigmas[t % len(sigmas)])
              for t in range(steps)]
    qs = [synth.make_q(cfg, n_q, step=t) for t in range(steps)]
    d_in = [(dev(li.target_logits), dev(li.draft_logits), dev(li.draft_tokens), dev(li.u_accept),
             dev(li.u_sample), dev_bf16(q)) for li, q in zip(inputs, qs)]

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
    sl0 = sl.clone()
    for t in range(steps):
        tl, dl, x, ua, us, q = d_in[t]
        sv.spec_verify_attn(q, o[t], pool, bt, sl, g, d_cq, gmax, max_len, ws_a, device_status=status)
        sv.spec_accept_sample(tl, dl, x, ua, us, cfg.temperature, g, d_cq, d_cd, gmax, n_acc, toks[t], ws_s,
                              device_status=status)
        sv.gamma_tune_update(n_acc, gbar, g, sl, d_cq, d_cd, gcfg, trajectory=traj, accepted_log=n_log,
                             step=t, device_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return dict(kv=kv, inputs=inputs, qs=qs, cu_q=cu_q, cu_d=cu_d, sl0=sl0.cpu().numpy(),
                toks=toks.cpu().numpy(), n_log=n_log.cpu().numpy(), traj=traj.cpu().numpy(),
                o=o, gbar=gbar.cpu().numpy(), sl=sl.cpu().numpy())


def replay_with_oracle(cfg, run, steps, gamma0, gcfg, check_attn_steps=()):
    B, gmax = cfg.batch, cfg.gamma_max
    gbar, g, _, _ = oracle.gamma_tune_init(B, gamma0, gmax, True)
    sl = run["sl0"].copy()
    flagged = 0
    scale = float(np.float32(cfg.head_dim ** -0.5))
    for t in range(steps):
        li = run["inputs"][t]
        gpu = AcceptOut(run["n_log"][t], run["toks"][t], None, None, None, 0, 0)
        ref, n_pos, n_tok = compare_accept(gpu, li, cfg.temperature, g, run["cu_q"], run["cu_d"], gmax)
        flagged += n_pos + n_tok
        if t in check_attn_steps:
            o_ref, _ = oracle.verify_attn(run["qs"][t], run["kv"].k_pool, run["kv"].v_pool, run["kv"].strides,
                                          run["kv"].block_table, sl, g, run["cu_q"], cfg.hq, cfg.hkv,
                                          cfg.page_size, scale)
            o_gpu = synth.bf16_to_f32(bits_of(run["o"][t])).astype(np.float64)
            for b in range(B):
                rows = slice(run["cu_q"][b], run["cu_q"][b] + g[b] + 1)
                assert np.abs(o_gpu[rows] - o_ref[rows]).max() <= ATTN_ATOL
        # follow the device through near ties (compare_accept has already checked legality)
        gbar, g, sl, _, _ = oracle.gamma_tune_update(run["n_log"][t], gbar, g, sl, gcfg.eta, gcfg.delta,
                                                     gcfg.gamma_min, gcfg.gamma_max, gcfg.mode, True)
        np.testing.assert_array_equal(run["traj"][t], g)
    np.testing.assert_array_equal(run["gbar"].view(np.int64), gbar.view(np.int64))
    np.testing.assert_array_equal(run["sl"], sl)
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


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_c4_alternating_regimes_reduced(T):
    # vicuna-13B shape at reduced batch / heads / context; acceptance regime flips every 8 steps
    cfg = synth.scaled(synth.CONFIGS["c4"], batch=8, hq=4, hkv=4, ctx_lo=600, ctx_hi=600, temperature=T)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, 12, sv.SV_GT_PROPOSED, True)
    steps = 32
    sig = [0.1] * 8 + [3.0] * 8
    run = run_loop(cfg, steps, 4, gcfg, sig, 600)
    replay_with_oracle(cfg, run, steps, 4, gcfg, check_attn_steps=(5, 20))
    easy = run["traj"][4:8].mean()
    hard = run["traj"][12:16].mean()
    assert easy > hard                                  # expands when drafts are accepted, contracts otherwise


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
