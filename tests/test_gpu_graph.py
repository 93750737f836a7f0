"""The verify step captured once into a CUDA graph and replayed: the library allocates nothing, reads nothing back
and keeps its state on the device, so a caller can turn the launch-bound small steps into one graph launch.  Four
replays with fresh inputs in the same buffers (the controller's state carries over) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import DEV, AcceptOut, bits_of, compare_accept, dev, dev_bf16, workspace

pytestmark = pytest.mark.gpu

ATTN_ATOL = 2e-2


def test_captured_step_replays_against_the_oracle():
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=2, gamma_max=6, gamma_lo=6, gamma_hi=6, ctx_lo=700, ctx_hi=700)
    B, gmax, steps, L0 = cfg.batch, cfg.gamma_max, 4, 700
    gcfg = sv.GammaConfig(0.5, 2.0, 1, gmax, sv.SV_GT_PROPOSED, True)
    cu_q, cu_d = synth.padded_offsets(B, gmax)
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    full = np.full(B, gmax, np.int32)
    seq_len0 = np.full(B, L0, np.int32)
    kv = synth.make_kv(cfg, seq_len0, reserve_tokens=steps * (gmax + 1))
    k, v = dev_bf16(kv.k_pool), dev_bf16(kv.v_pool)
    pool = sv.spec_kv_pool_register(k, v)
    bt = dev(kv.block_table)
    max_len = L0 + steps * (gmax + 1)
    inputs = [synth.make_logits(cfg, full, cu_q, cu_d, step=t, sigma_noise=0.6) for t in range(steps)]
    qs = [synth.make_q(cfg, n_q, step=t) for t in range(steps)]

    # fixed buffers: the graph holds their addresses
    q = torch.zeros((n_q, cfg.hq, cfg.head_dim), dtype=torch.bfloat16, device=DEV)
    o = torch.zeros_like(q)
    tl = torch.zeros((n_q, cfg.vocab), device=DEV)
    dl = torch.zeros((n_d, cfg.vocab), device=DEV)
    x = torch.zeros(n_d, dtype=torch.int32, device=DEV)
    ua, us = torch.zeros(n_d, device=DEV), torch.zeros(B, device=DEV)
    n_acc = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = torch.zeros((B, gmax + 1), dtype=torch.int32, device=DEV)
    gbar = torch.zeros(B, dtype=torch.float64, device=DEV)
    g = torch.zeros(B, dtype=torch.int32, device=DEV)
    sl = dev(seq_len0)
    d_cq = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    d_cd = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws_a = workspace(sv.spec_verify_attn_workspace_bytes(B, gmax, cfg.hq, cfg.hkv, cfg.head_dim, max_len))
    ws_s = workspace(sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab))

    def load(t):
        q.copy_(dev_bf16(qs[t]))
        li = inputs[t]
        tl.copy_(dev(li.target_logits)); dl.copy_(dev(li.draft_logits)); x.copy_(dev(li.draft_tokens))
        ua.copy_(dev(li.u_accept)); us.copy_(dev(li.u_sample))

    def step(stream):
        sv.spec_verify_attn(q, o, pool, bt, sl, g, d_cq, gmax, max_len, ws_a, device_status=status, stream=stream)
        sv.spec_accept_sample(tl, dl, x, ua, us, cfg.temperature, g, d_cq, d_cd, gmax, n_acc, toks, ws_s,
                              device_status=status, stream=stream)
        sv.gamma_tune_update(n_acc, gbar, g, sl, d_cq, d_cd, gcfg, device_status=status, stream=stream)

    side = torch.cuda.Stream()
    # one uncaptured step first (occupancy and attribute queries of the first call), then the state is set up
    load(0)
    sv.gamma_tune_init(gbar, g, d_cq, d_cd, gcfg, 3)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        step(side)
    torch.cuda.synchronize()
    sv.gamma_tune_init(gbar, g, d_cq, d_cd, gcfg, 3)
    sl.copy_(dev(seq_len0))
    torch.cuda.synchronize()

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    torch.cuda.synchronize()
    # the capture itself ran nothing
    assert sl.cpu().numpy().tolist() == seq_len0.tolist()

    o_gbar, o_g, _, _ = oracle.gamma_tune_init(B, 3, gmax, True)
    o_sl = seq_len0.copy()
    scale = float(np.float32(cfg.head_dim ** -0.5))
    for t in range(steps):
        load(t)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        gpu = AcceptOut(n_acc.cpu().numpy(), toks.cpu().numpy(), None, None, None, 0, 0)
        compare_accept(gpu, inputs[t], cfg.temperature, o_g, cu_q, cu_d, gmax)
        o_ref, _ = oracle.verify_attn(qs[t], kv.k_pool, kv.v_pool, kv.strides, kv.block_table, o_sl, o_g, cu_q,
                                      cfg.hq, cfg.hkv, cfg.page_size, scale)
        o_gpu = synth.bf16_to_f32(bits_of(o)).astype(np.float64)
        for b in range(B):
            rows = slice(cu_q[b], cu_q[b] + o_g[b] + 1)
            assert np.abs(o_gpu[rows] - o_ref[rows]).max() <= ATTN_ATOL
        o_gbar, o_g, o_sl, _, _ = oracle.gamma_tune_update(gpu.n_accepted, o_gbar, o_g, o_sl, gcfg.eta, gcfg.delta,
                                                           gcfg.gamma_min, gcfg.gamma_max, gcfg.mode, True)
        np.testing.assert_array_equal(g.cpu().numpy(), o_g)
        np.testing.assert_array_equal(sl.cpu().numpy(), o_sl)
    np.testing.assert_array_equal(gbar.cpu().numpy().view(np.int64), o_gbar.view(np.int64))
