"""spec_draft_step (one drafting step with the confidence stop, paper Section 4.2) on the GPU against the
oracle: tokens, n_drafted and active bit-exact except where the oracle flags a draw within 1e-9 of a CDF edge
or a confidence within 1e-6 of tau (there the device's own answer must be the other legal one, and the oracle's
state follows it); confidences to 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import DEV, dev, workspace

pytestmark = pytest.mark.gpu


class Loop:
    """Drafting state held on both sides."""

    def __init__(self, gamma, gamma_max, V, active=None):
        self.gamma = np.asarray(gamma, np.int32)
        self.B, self.gmax, self.V = len(self.gamma), gamma_max, V
        self.cu_d = np.zeros(self.B + 1, np.int32)
        self.cu_d[1:] = np.cumsum(self.gamma)
        n_d = max(int(self.cu_d[-1]), 1)
        act = np.ones(self.B, np.int32) if active is None else np.asarray(active, np.int32)
        self.ref = (np.zeros(self.B, np.int32), act.copy(), np.full(n_d, -1, np.int32), np.full(n_d, np.nan))
        self.n = dev(self.ref[0].copy())
        self.act = dev(act.copy())
        self.tok = torch.full((n_d,), -1, dtype=torch.int32, device=DEV)
        self.top = torch.full((n_d,), float("nan"), dtype=torch.float64, device=DEV)
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)
        self.ws = workspace(sv.spec_draft_step_workspace_bytes(self.B, V))
        self.g_dev, self.cu_dev = dev(self.gamma), dev(self.cu_d)
        self.flagged = 0

    def step(self, logits, T, tau, u, T_per_seq=None, bf16=False):
        """One step on the device and in the oracle; compares and lets the oracle follow flagged decisions."""
        ldt = torch.bfloat16 if bf16 else torch.float32      # bf16: the values are bf16-representable already
        dl = dev(np.ascontiguousarray(logits, np.float32)).to(ldt)
        tps = dev(np.asarray(T_per_seq, np.float32)) if T_per_seq is not None else None
        sv.spec_draft_step(dl, float(T), float(tau), dev(np.asarray(u, np.float32)), self.g_dev, self.cu_dev,
                           self.gmax, self.n, self.act, self.tok, self.ws, top_prob=self.top,
                           device_status=self.status, temperature_per_seq=tps)
        torch.cuda.synchronize()
        n0 = self.ref[0].copy()
        was = self.ref[1].copy()
        alt, sflag, cflag = oracle.draft_step(logits, T_per_seq if T_per_seq is not None else T, tau, u, self.gamma,
                                              self.cu_d, *self.ref)
        n_g, act_g = self.n.cpu().numpy(), self.act.cpu().numpy()
        tok_g, top_g = self.tok.cpu().numpy(), self.top.cpu().numpy()
        n_r, act_r, tok_r, top_r = self.ref
        assert (n_g == n_r).all()
        for b in range(self.B):
            if not was[b] or n0[b] >= self.gamma[b]:
                continue
            pos = self.cu_d[b] + n0[b]
            if tok_g[pos] != tok_r[pos]:
                assert sflag[b] and tok_g[pos] == alt[b], \
                    f"sequence {b}: token {tok_g[pos]} vs oracle {tok_r[pos]} (alt {alt[b]}, flag {sflag[b]})"
                tok_r[pos] = tok_g[pos]
                self.flagged += 1
            assert abs(top_g[pos] / top_r[pos] - 1.0) <= 1e-5
            if act_g[b] != act_r[b]:
                assert cflag[b], f"sequence {b}: active {act_g[b]} vs oracle {act_r[b]}, confidence {top_r[pos]}"
                assert act_g[b] == int(top_g[pos] >= tau and n_g[b] < self.gamma[b])
                act_r[b] = act_g[b]
                self.flagged += 1
        # nothing else was touched
        same = np.ones(len(tok_r), bool)
        assert (tok_g[same] == tok_r[same]).all()
        assert (np.isnan(top_g) == np.isnan(top_r)).all()
        assert (act_g == act_r).all()
        return n_g, act_g


def rows_for(cfg, B, step, sigmas=None):
    """B rows of draft logits of the configuration's distribution."""
    g = np.ones(B, np.int32)
    cu_q, cu_d = synth.prefix(g)
    li = synth.make_logits(synth.scaled(cfg, batch=B), g, cu_q, cu_d, step, row_sigmas=sigmas)
    return li.draft_logits


@pytest.mark.parametrize("name,B,gamma_max", [("c1", 3, 4), ("c2", 2, 8), ("c3", 6, 10), ("c5", 5, 6)])
def test_drafting_loop_on_config_shapes(name, B, gamma_max):
    cfg = synth.CONFIGS[name]
    r = np.random.default_rng(cfg.seed + 77)
    gamma = r.integers(0, gamma_max + 1, size=B).astype(np.int32)
    gamma[0] = gamma_max
    loop = Loop(gamma, gamma_max, cfg.vocab, active=(gamma > 0).astype(np.int32))
    T = cfg.temperature if cfg.temperature > 0 else 1.0
    # tau at the median top probability of such rows, so that both outcomes occur
    probe = rows_for(cfg, 8, 999)
    _, top, _ = oracle.draft_stop(probe, T, 0.0, np.ones(8, np.int32), np.arange(9, dtype=np.int32))
    tau = float(np.median(top))
    for i in range(gamma_max):
        _, act = loop.step(rows_for(cfg, B, i), T, tau, r.random(B).astype(np.float32))
    assert (act == 0).all()
    assert int(loop.status.item()) == 0
    assert loop.flagged <= 1
    n = loop.n.cpu().numpy()
    assert (n <= gamma).all() and (n[gamma > 0] >= 1).all()
    assert (n < gamma).any() or gamma_max < 3          # the threshold did stop someone early


def test_ragged_vocabulary_per_sequence_temperature_and_unaligned_rows():
    r = np.random.default_rng(3)
    B, V, gmax = 9, 1003, 5                      # 1003: no 128-bit loads, a ragged last slice
    gamma = np.array([5, 1, 3, 5, 2, 5, 4, 5, 5], np.int32)
    T = np.array([0.3, 0.7, 1.0, 1.0, 1.5, 2.5, 0.0, 4.0, 0.05], np.float32)
    loop = Loop(gamma, gmax, V)
    for i in range(gmax):
        d = (r.standard_normal((B, V)) * r.choice([0.5, 2.0, 5.0], size=(B, 1))).astype(np.float32)
        loop.step(d, 1.0, 0.02, r.random(B).astype(np.float32), T_per_seq=T)
    assert int(loop.status.item()) == 0
    assert loop.flagged == 0


def test_bf16_logits():
    cfg = synth.CONFIGS["c3"]
    r = np.random.default_rng(12)
    B, gmax = 4, 4
    loop = Loop(np.full(B, gmax, np.int32), gmax, cfg.vocab)
    for i in range(gmax):
        d = rows_for(cfg, B, 40 + i)
        d16 = torch.from_numpy(d).to(torch.bfloat16).to(torch.float32).numpy()     # the values both sides see
        loop.step(d16, 0.8, 0.01, r.random(B).astype(np.float32), bf16=True)
    assert int(loop.status.item()) == 0


def test_greedy_ties_take_the_lowest_index():
    V = 5000
    d = np.zeros((3, V), np.float32)
    d[0, [4999, 17, 3000]] = 2.0
    d[1, 4096] = 1.0
    d[2] = -np.inf
    d[2, 4999] = -3.0
    loop = Loop([2, 2, 2], 2, V)
    loop.step(d, 0.0, 0.9, np.zeros(3, np.float32))
    assert list(loop.tok.cpu().numpy()[[0, 2, 4]]) == [17, 4096, 4999]
    assert list(loop.act.cpu().numpy()) == [1, 1, 1]          # a greedy draft's confidence is one


def test_same_counts_as_the_block_form():
    """Steps over the rows of a block end with the n_drafted spec_draft_stop gives for the block."""
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=6)
    r = np.random.default_rng(21)
    gamma = np.array([10, 7, 10, 3, 10, 9], np.int32)
    cu_q, cu_d = synth.prefix(gamma)
    sig = synth.mixture_rows(cfg, int(cu_q[-1]), 0, 0.4)
    block = synth.make_logits(cfg, gamma, cu_q, cu_d, 0, row_sigmas=sig).draft_logits
    T, tau = 0.9, 0.03
    loop = Loop(gamma, 10, cfg.vocab)
    for i in range(10):
        d = np.zeros((6, cfg.vocab), np.float32)
        for b in range(6):
            if i < gamma[b]:
                d[b] = block[cu_d[b] + i]
        loop.step(d, T, tau, r.random(6).astype(np.float32))
    n_block = torch.zeros(6, dtype=torch.int32, device=DEV)
    ws = workspace(sv.spec_draft_stop_workspace_bytes(6, 10, cfg.vocab))
    sv.spec_draft_stop(dev(block), T, tau, dev(gamma), dev(cu_d), 10, n_block, ws)
    torch.cuda.synchronize()
    assert (loop.n.cpu().numpy() == n_block.cpu().numpy()).all()
    assert (n_block.cpu().numpy() < gamma).any()


def test_nonfinite_rows_are_reported_and_end_the_drafting():
    V = 3000
    r = np.random.default_rng(4)
    d = r.standard_normal((4, V)).astype(np.float32)
    d[1, 1234] = np.nan
    d[2, 77] = np.inf
    B = 4
    gamma, cu_d = dev(np.full(B, 3, np.int32)), dev(np.arange(B + 1, dtype=np.int32) * 3)
    n = torch.zeros(B, dtype=torch.int32, device=DEV)
    act = torch.ones(B, dtype=torch.int32, device=DEV)
    tok = torch.full((3 * B,), -5, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = workspace(sv.spec_draft_step_workspace_bytes(B, V))
    sv.spec_draft_step(dev(d), 1.0, 0.0, dev(np.full(B, 0.5, np.float32)), gamma, cu_d, 3, n, act, tok, ws,
                       device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & sv.SV_DEV_NONFINITE
    assert list(act.cpu().numpy()) == [1, 0, 0, 1]
    t = tok.cpu().numpy()
    assert t[3] == -1 and t[6] == -1 and t[0] >= 0 and t[9] >= 0
    assert list(n.cpu().numpy()) == [1, 1, 1, 1]
    # the untouched sequences' tokens are the oracle's
    st = (np.zeros(2, np.int32), np.ones(2, np.int32), np.full(2, -1, np.int32), np.full(2, np.nan))
    oracle.draft_step(d[[0, 3]], 1.0, 0.0, np.full(2, 0.5, np.float32), np.ones(2, np.int32),
                      np.arange(3, dtype=np.int32), *st)
    assert t[0] == st[2][0] and t[9] == st[2][1]
    # greedy: a NaN in the row
    n.zero_(); act.fill_(1); status.zero_()
    sv.spec_draft_step(dev(d), 0.0, 0.0, None, gamma, cu_d, 3, n, act, tok, ws, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & sv.SV_DEV_NONFINITE
    assert list(act.cpu().numpy()) == [1, 0, 1, 1]            # +inf is a legal argmax
    assert tok.cpu().numpy()[6] == 77


def test_inactive_and_finished_sequences_are_not_touched():
    V = 2048
    r = np.random.default_rng(9)
    gamma = np.array([2, 2, 0, 2], np.int32)
    loop = Loop(gamma, 2, V, active=[1, 0, 1, 1])
    n, act = loop.step(r.standard_normal((4, V)).astype(np.float32), 1.0, 0.0, r.random(4).astype(np.float32))
    assert list(n) == [1, 0, 0, 1] and list(act) == [1, 0, 0, 1]
    n, act = loop.step(r.standard_normal((4, V)).astype(np.float32), 1.0, 0.0, r.random(4).astype(np.float32))
    assert list(n) == [2, 0, 0, 2] and list(act) == [0, 0, 0, 0]
    before = loop.tok.cpu().numpy().copy()
    n, act = loop.step(np.full((4, V), np.nan, np.float32), 1.0, 0.0, r.random(4).astype(np.float32))
    assert (loop.tok.cpu().numpy() == before).all() and int(loop.status.item()) == 0     # rows were not read


def test_host_errors():
    B, V = 2, 512
    d = torch.zeros((B, V), device=DEV)
    g = dev(np.ones(B, np.int32))
    cu = dev(np.arange(B + 1, dtype=np.int32))
    n = torch.zeros(B, dtype=torch.int32, device=DEV)
    act = torch.ones(B, dtype=torch.int32, device=DEV)
    tok = torch.zeros(B, dtype=torch.int32, device=DEV)
    u = torch.zeros(B, device=DEV)
    ws = workspace(sv.spec_draft_step_workspace_bytes(B, V))
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.spec_draft_step(d, 1.0, 1.5, u, g, cu, 1, n, act, tok, ws)
    assert e.value.status == sv.SV_EINVAL
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.spec_draft_step(d, 1.0, 0.5, None, g, cu, 1, n, act, tok, ws)          # sampling without uniforms
    assert e.value.status == sv.SV_EINVAL
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.spec_draft_step(d, 1.0, 0.5, u, g, cu, 1, n, act, tok, ws[:256])
    assert e.value.status == sv.SV_EWORKSPACE
    assert sv.spec_draft_step_workspace_bytes(0, V) == 0
    torch.cuda.synchronize()
    assert list(n.cpu().numpy()) == [0, 0]


def test_one_step_at_the_largest_size():
    """Batch 128 over the 128256-token vocabulary of c5, the launch shape a drafting loop of that workload has."""
    cfg = synth.CONFIGS["c5"]
    r = np.random.default_rng(cfg.seed)
    B = cfg.batch
    sig = synth.mixture_rows(cfg, 2 * B, 0, 0.5)          # one per target row of the generator
    d = rows_for(cfg, B, 3, sigmas=sig)
    loop = Loop(np.full(B, 2, np.int32), 2, cfg.vocab)
    _, top, _ = oracle.draft_stop(d, 1.0, 0.0, np.ones(B, np.int32), np.arange(B + 1, dtype=np.int32))
    n, act = loop.step(d, 1.0, float(np.median(top)), r.random(B).astype(np.float32))
    assert int(loop.status.item()) == 0
    assert 0 < int(act.sum()) < B and (n == 1).all()


def test_drafting_loop_feeds_the_verify_step_without_a_host_round_trip():
    """Three speculative steps of a small batch, all state on the device: the draft tokens of every block come
    from a loop of spec_draft_step calls (strided views of the block's draft rows, no copy), spec_accept_sample
    reads them where they were written with n_drafted as its draft lengths, and the controller is told both.
    Nothing is read back until the end; the oracle then takes the same steps."""
    import dataclasses
    from tests.harness import AcceptOut, compare_accept
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=3, gamma_max=6, gamma_lo=6, gamma_hi=6)
    B, gmax, V, T, tau, steps = cfg.batch, cfg.gamma_max, cfg.vocab, 1.0, 0.012, 3
    gcfg = sv.GammaConfig(0.5, 2.0, 1, gmax, sv.SV_GT_PROPOSED, True)
    cu_q, cu_d = synth.padded_offsets(B, gmax)
    full = np.full(B, gmax, np.int32)
    rng = np.random.default_rng(31)
    inputs = [synth.make_logits(cfg, full, cu_q, cu_d, step=t, sigma_noise=0.7, temperature=T) for t in range(steps)]
    u_draft = [rng.random((gmax, B)).astype(np.float32) for _ in range(steps)]

    gbar = torch.zeros(B, dtype=torch.float64, device=DEV)
    g = torch.zeros(B, dtype=torch.int32, device=DEV)
    sl = dev(np.full(B, 500, np.int32))
    d_cq = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    d_cd = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    sv.gamma_tune_init(gbar, g, d_cq, d_cd, gcfg, 4)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    n_dr = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    act = torch.zeros(B, dtype=torch.int32, device=DEV)
    x = torch.full((steps, B * gmax), -1, dtype=torch.int32, device=DEV)
    n_acc = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    toks = torch.zeros((steps, B, gmax + 1), dtype=torch.int32, device=DEV)
    traj = torch.zeros((steps, B), dtype=torch.int32, device=DEV)
    ws_p = workspace(sv.spec_draft_step_workspace_bytes(B, V))
    ws_s = workspace(sv.spec_accept_sample_workspace_bytes(B, gmax, V))
    d_in = [(dev(li.target_logits), dev(li.draft_logits), dev(li.u_accept), dev(li.u_sample)) for li in inputs]
    d_u = [dev(u) for u in u_draft]
    for t in range(steps):
        tl, dl, ua, us = d_in[t]
        act.fill_(1)
        rows = dl.view(B, gmax, V)
        for i in range(gmax):
            sv.spec_draft_step(rows[:, i], T, tau, d_u[t][i], g, d_cd, gmax, n_dr[t], act, x[t], ws_p,
                               device_status=status)
        sv.spec_accept_sample(tl, dl, x[t], ua, us, T, n_dr[t], d_cq, d_cd, gmax, n_acc[t], toks[t], ws_s,
                              device_status=status)
        sv.gamma_tune_update(n_acc[t], gbar, g, sl, d_cq, d_cd, gcfg, trajectory=traj, step=t,
                             device_status=status, n_drafted=n_dr[t])
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    n_dr, x, n_acc, toks, traj = (a.cpu().numpy() for a in (n_dr, x, n_acc, toks, traj))

    o_gbar, o_g, _, _ = oracle.gamma_tune_init(B, 4, gmax, True)
    o_sl = np.full(B, 500, np.int32)
    stopped_early = 0
    for t in range(steps):
        li = inputs[t]
        st = (np.zeros(B, np.int32), np.ones(B, np.int32), np.full(B * gmax, -1, np.int32), np.full(B * gmax, np.nan))
        for i in range(gmax):
            d = li.draft_logits.reshape(B, gmax, V)[:, i]
            alt, sflag, cflag = oracle.draft_step(d, T, tau, u_draft[t][i], o_g, cu_d, *st)
            assert not sflag.any() and not cflag.any()          # these seeds meet no near tie
        np.testing.assert_array_equal(n_dr[t], st[0])
        np.testing.assert_array_equal(x[t], st[2])
        stopped_early += int((st[0] < o_g).sum())
        gpu = AcceptOut(n_acc[t], toks[t], None, None, None, 0, 0)
        compare_accept(gpu, dataclasses.replace(li, draft_tokens=st[2]), T, st[0], cu_q, cu_d, gmax)
        o_gbar, o_g, o_sl, _, _ = oracle.gamma_tune_update(n_acc[t], o_gbar, o_g, o_sl, gcfg.eta, gcfg.delta,
                                                           gcfg.gamma_min, gcfg.gamma_max, gcfg.mode, True,
                                                           n_drafted=st[0])
        np.testing.assert_array_equal(traj[t], o_g)
    assert stopped_early > 0
    np.testing.assert_array_equal(gbar.cpu().numpy().view(np.int64), o_gbar.view(np.int64))
    np.testing.assert_array_equal(sl.cpu().numpy(), o_sl)
