"""spec_draft_stop (GammaTune+ early stop) on the GPU against the oracle: n_drafted bit-exact except
where the oracle flags a confidence within 1e-6 of tau, confidences to 1e-5 relative; and the
controller's bookkeeping after an early stop."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import DEV, dev, workspace

pytestmark = pytest.mark.gpu


def run_gpu(draft_logits, T, tau, gamma, cu_d, gamma_max, T_per_seq=None, bf16=False):
    B = len(gamma)
    n_d = int(cu_d[-1])
    V = draft_logits.shape[1]
    ldt = torch.bfloat16 if bf16 else torch.float32      # bf16: the values are bf16-representable already
    dl = dev(draft_logits).to(ldt) if n_d > 0 else torch.zeros((1, V), dtype=ldt, device=DEV)
    n = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    top = torch.full((max(n_d, 1),), float("nan"), dtype=torch.float64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = workspace(sv.spec_draft_stop_workspace_bytes(B, gamma_max, V))
    tps = dev(np.asarray(T_per_seq, np.float32)) if T_per_seq is not None else None
    sv.spec_draft_stop(dl, float(T), float(tau), dev(gamma), dev(cu_d), gamma_max, n, ws, top_prob=top,
                       device_status=status, temperature_per_seq=tps)
    torch.cuda.synchronize()
    return n.cpu().numpy(), top.cpu().numpy()[:n_d], int(status.item())


def check(draft_logits, T, tau, gamma, cu_d, gamma_max, T_per_seq=None, bf16=False):
    Tref = T_per_seq if T_per_seq is not None else T
    n_gpu, top_gpu, status = run_gpu(draft_logits, T, tau, gamma, cu_d, gamma_max, T_per_seq, bf16)
    assert status == 0
    n_ref, top_ref, flag = oracle.draft_stop(draft_logits, Tref, tau, gamma, cu_d)
    if len(top_ref):
        assert np.abs(top_gpu / top_ref - 1.0).max() <= 1e-5
    flagged = 0
    for b in range(len(gamma)):
        if n_gpu[b] == n_ref[b]:
            continue
        # the first decision that differs is at position min(n) - 1; it must be a flagged near tie,
        # and the device's own count must follow from its own decisions
        i = int(min(n_gpu[b], n_ref[b])) - 1
        assert flag[cu_d[b] + i], f"sequence {b}: {n_gpu[b]} vs oracle {n_ref[b]}, position {i} is no near tie"
        conf = top_gpu[cu_d[b]:cu_d[b] + gamma[b]]
        below = np.flatnonzero(conf < tau)
        assert n_gpu[b] == (min(gamma[b], below[0] + 1) if len(below) else gamma[b])
        flagged += 1
    return n_gpu, n_ref, top_ref, flagged


def logits_case(cfg, gamma=None, step=0):
    _, g = synth.draw_lengths(cfg, step)
    if gamma is not None:
        g = np.asarray(gamma, np.int32)
    cu_q, cu_d = synth.prefix(g)
    li = synth.make_logits(cfg, g, cu_q, cu_d, step)
    return li.draft_logits, g, cu_d


@pytest.mark.parametrize("name,batch", [("c1", None), ("c2", None), ("c3", 4), ("c5", 5)])
def test_config_shapes(name, batch):
    cfg = synth.CONFIGS[name]
    if batch:
        cfg = synth.scaled(cfg, batch=batch)
    d, g, cu_d = logits_case(cfg)
    T = cfg.temperature
    # a threshold at the median confidence, so that about half of the positions would stop the draft
    _, top, _ = oracle.draft_stop(d, T, 0.0, g, cu_d)
    for tau in (float(np.median(top)), float(np.quantile(top, 0.1)), float(top.max()) * 1.01):
        n_gpu, n_ref, _, _ = check(d, T, min(tau, 1.0), g, cu_d, cfg.gamma_max)
    assert (n_gpu <= g).all() and (n_gpu >= np.minimum(g, 1)).all()


@pytest.mark.parametrize("V", [1, 2, 3, 5, 127, 129, 1001, 4099])
def test_small_and_odd_vocabularies(V):
    rng = np.random.default_rng(V)
    gamma = np.array([3, 0, 5, 1, 4], np.int32)
    cu_d = np.concatenate([[0], np.cumsum(gamma)]).astype(np.int32)
    d = (rng.standard_normal((int(cu_d[-1]), V)) * 2.0).astype(np.float32)
    _, top, _ = oracle.draft_stop(d, 1.0, 0.0, gamma, cu_d)
    check(d, 1.0, float(np.median(top)), gamma, cu_d, 5)


@pytest.mark.parametrize("V", [3, 8, 1001, 32000])
def test_bf16_logits(V):
    # draft rows stored as bf16: widened exactly on the device, so the oracle sees the same values
    rng = np.random.default_rng(100 + V)
    gamma = np.array([3, 0, 5, 1, 4], np.int32)
    cu_d = np.concatenate([[0], np.cumsum(gamma)]).astype(np.int32)
    d = (rng.standard_normal((int(cu_d[-1]), V)) * 2.0).astype(np.float32)
    d = synth.bf16_to_f32(synth.bf16_bits(d)).reshape(d.shape)
    _, top, _ = oracle.draft_stop(d, 1.0, 0.0, gamma, cu_d)
    check(d, 1.0, float(np.median(top)), gamma, cu_d, 5, bf16=True)


def test_longest_draft_blocks():
    # gamma up to the maximum of 64 with several slices per row: the decision walks the positions in passes
    rng = np.random.default_rng(21)
    gamma = np.array([64, 0, 33, 64], np.int32)
    cu_d = np.concatenate([[0], np.cumsum(gamma)]).astype(np.int32)
    d = (rng.standard_normal((int(cu_d[-1]), 9000)) * 2.0).astype(np.float32)
    _, top, _ = oracle.draft_stop(d, 1.0, 0.0, gamma, cu_d)
    for q in (0.0, 0.02, 0.5):                               # never, late and early stops
        n_gpu, n_ref, _, _ = check(d, 1.0, float(np.quantile(top, q)) if q > 0 else 0.0, gamma, cu_d, 64)
    assert n_ref[0] < 64 and n_ref[1] == 0


def test_row_stride_and_per_sequence_temperatures():
    rng = np.random.default_rng(11)
    gamma = np.array([4, 4, 2, 4], np.int32)
    cu_d = np.concatenate([[0], np.cumsum(gamma)]).astype(np.int32)
    V, stride = 3001, 3008
    full = (rng.standard_normal((int(cu_d[-1]), stride)) * 2.5).astype(np.float32)
    T = np.array([1.0, 0.0, 0.4, 2.0], np.float32)           # sequence 1 drafts greedily: never stops
    full[:, V:] = 50.0                                        # poison in the padding
    n = torch.zeros(4, dtype=torch.int32, device=DEV)
    top = torch.zeros(int(cu_d[-1]), dtype=torch.float64, device=DEV)
    ws = workspace(sv.spec_draft_stop_workspace_bytes(4, 4, stride))
    ref_n, ref_top, _ = oracle.draft_stop(np.ascontiguousarray(full[:, :V]), T, 0.01, gamma, cu_d)
    # the padded buffer goes in whole; the true vocabulary is set by hand
    p = sv.draft_stop_params(dev(full), 1.0, 0.01, dev(gamma), dev(cu_d), 4, n, top_prob=top,
                             temperature_per_seq=dev(T))
    p.vocab = V
    import ctypes as C
    assert sv.load().spec_draft_stop(C.byref(p), ws.data_ptr(), ws.numel(), None) == 0
    torch.cuda.synchronize()
    np.testing.assert_array_equal(n.cpu().numpy(), ref_n)
    assert np.abs(top.cpu().numpy() / ref_top - 1.0).max() <= 1e-5
    assert ref_n[1] == 4


def test_threshold_extremes():
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=3, vocab=4000)
    d, g, cu_d = logits_case(cfg)
    n, _, _ = run_gpu(d, 1.0, 0.0, g, cu_d, cfg.gamma_max)
    np.testing.assert_array_equal(n, g)                       # nothing is below zero
    n, _, _ = run_gpu(d, 1.0, 1.0, g, cu_d, cfg.gamma_max)
    np.testing.assert_array_equal(n, np.minimum(g, 1))        # every confidence is below one


def test_host_errors_and_bad_gamma_status():
    d = dev(np.zeros((4, 64), np.float32))
    g, cd = dev(np.array([4], np.int32)), dev(np.array([0, 4], np.int32))
    n = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = workspace(sv.spec_draft_stop_workspace_bytes(1, 4, 64))
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.spec_draft_stop(d, 1.0, 1.5, g, cd, 4, n, ws)
    assert e.value.status == sv.SV_EINVAL
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.spec_draft_stop(d, 1.0, 0.5, g, cd, 4, n, torch.empty(16, dtype=torch.uint8, device=DEV))
    assert e.value.status == sv.SV_EWORKSPACE
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sv.spec_draft_stop(d, 1.0, 0.5, dev(np.array([9], np.int32)), cd, 4, n, ws, device_status=status)
    torch.cuda.synchronize()
    assert status.item() & sv.SV_DEV_BAD_GAMMA


def test_step_with_early_stop_feeds_the_controller():
    """draft stop -> accept with n_drafted as its gamma -> controller update with both, all on the
    device with fixed row slabs; the oracle replays the same chain."""
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=6, vocab=8000, gamma_lo=10, gamma_hi=10)
    B, gmax = cfg.batch, cfg.gamma_max
    gamma = np.full(B, gmax, np.int32)
    cu_q, cu_d = synth.padded_offsets(B, gmax)
    li = synth.make_logits(cfg, gamma, cu_q, cu_d)
    T = cfg.temperature
    _, top, _ = oracle.draft_stop(li.draft_logits, T, 0.0, gamma, cu_d)
    tau = float(np.quantile(top, 0.15))
    seq_len = np.full(B, 500, np.int32)
    # device
    d_gamma, d_cq, d_cd = dev(gamma), dev(cu_q), dev(cu_d)
    n_dr = torch.zeros(B, dtype=torch.int32, device=DEV)
    sv.spec_draft_stop(dev(li.draft_logits), T, tau, d_gamma, d_cd, gmax, n_dr,
                       workspace(sv.spec_draft_stop_workspace_bytes(B, gmax, cfg.vocab)))
    n_acc = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = torch.zeros((B, gmax + 1), dtype=torch.int32, device=DEV)
    sv.spec_accept_sample(dev(li.target_logits), dev(li.draft_logits), dev(li.draft_tokens), dev(li.u_accept),
                          dev(li.u_sample), T, n_dr, d_cq, d_cd, gmax, n_acc, toks,
                          workspace(sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab)))
    gbar = dev(gamma.astype(np.float64))
    sl = dev(seq_len)
    gcfg = sv.GammaConfig(0.5, 2.0, 1, gmax, sv.SV_GT_PROPOSED, True)
    sv.gamma_tune_update(n_acc, gbar, d_gamma, sl, d_cq, d_cd, gcfg, n_drafted=n_dr)
    torch.cuda.synchronize()
    # oracle
    o_n, _, flag = oracle.draft_stop(li.draft_logits, T, tau, gamma, cu_d)
    assert not flag.any()
    np.testing.assert_array_equal(n_dr.cpu().numpy(), o_n)
    assert (o_n < gamma).any() and (o_n > 1).any()            # the threshold bites, but not everywhere
    ref = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept, li.u_sample,
                               T, o_n, cu_q, cu_d, gmax)
    assert not ref.accept_flag.any()
    np.testing.assert_array_equal(n_acc.cpu().numpy(), ref.n_accepted)
    o_gbar, o_g, o_sl, o_cq, o_cd = oracle.gamma_tune_update(ref.n_accepted, gamma.astype(np.float64), gamma, seq_len,
                                                             0.5, 2.0, 1, gmax, oracle.MODE_GT_PROPOSED, True,
                                                             n_drafted=o_n)
    np.testing.assert_array_equal(gbar.cpu().numpy(), o_gbar)
    np.testing.assert_array_equal(d_gamma.cpu().numpy(), o_g)
    np.testing.assert_array_equal(sl.cpu().numpy(), o_sl)
    # a sequence whose draft stopped early never expands: its next gamma is at most ceil of the average
    early = o_n < gamma
    assert (o_g[early] <= gamma[early]).all()
