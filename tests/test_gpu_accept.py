"""spec_accept_sample on the GPU against the oracle: accepted counts and token ids bit-exact
(near ties as flagged by the oracle excepted), softmax sums to 1e-5 relative."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import DEV, check_accept, compare_accept, dev, run_accept_gpu
from tests.test_oracle_accept import chi2_p, draw_from, logits_of

pytestmark = pytest.mark.gpu


def case(cfg, gamma=None, padded=False, step=0, sigma=None, T=None):
    _, g = synth.draw_lengths(cfg, step)
    if gamma is not None:
        g = np.asarray(gamma, np.int32)
    cu_q, cu_d = synth.padded_offsets(cfg.batch, cfg.gamma_max) if padded else synth.prefix(g)
    li = synth.make_logits(cfg, g, cu_q, cu_d, step, sigma, T)
    return li, g, cu_q, cu_d


def test_config_c1_tiny():
    cfg = synth.CONFIGS["c1"]
    for step in range(8):
        li, g, cu_q, cu_d = case(cfg, step=step)
        check_accept(li, cfg.temperature, g, cu_q, cu_d, cfg.gamma_max)


@pytest.mark.parametrize("sigma", [0.3, 1.0, 2.0])
def test_config_c2_noise_sweep(sigma):
    cfg = synth.CONFIGS["c2"]
    for step, gam in enumerate([1, 3, 8, 5]):
        li, g, cu_q, cu_d = case(cfg, gamma=[gam], step=step, sigma=sigma)
        check_accept(li, cfg.temperature, g, cu_q, cu_d, cfg.gamma_max)


def test_config_c3_ragged_large_vocab():
    cfg = synth.CONFIGS["c3"]
    li, g, cu_q, cu_d = case(cfg)
    gpu, ref, n_pos, n_tok = check_accept(li, cfg.temperature, g, cu_q, cu_d, cfg.gamma_max)
    assert ref.n_accepted.sum() > 0            # the case exercises both accepts and rejections
    assert (ref.n_accepted < g).any()


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_config_c4_at_its_stated_size(T):
    # batch 64, V = 32000, gamma 1..12, both acceptance regimes (noise levels from the oracle's calibration
    # table: acceptance about 0.9 / 0.3), every sequence against the oracle
    cfg = synth.scaled(synth.CONFIGS["c4"], temperature=T)
    for sigma in {1.0: (0.25, 2.0), 0.0: (0.05, 1.0)}[T]:
        li, g, cu_q, cu_d = case(cfg, sigma=sigma, T=T, padded=True)
        check_accept(li, T, g, cu_q, cu_d, cfg.gamma_max)


def test_config_c5_shape_reduced_batch():
    cfg = synth.scaled(synth.CONFIGS["c5"], batch=6)
    li, g, cu_q, cu_d = case(cfg)
    check_accept(li, cfg.temperature, g, cu_q, cu_d, cfg.gamma_max)


@pytest.mark.parametrize("T", [0.0, 0.8])
def test_longest_draft_blocks(T):
    # gamma up to the library's maximum of 64 (129 rows per sequence): the decision kernel merges the rows
    # in several passes; small noise so that long runs of acceptances occur
    cfg = synth.VerifyConfig("max", 5, 8, 2, 128, 9000, 100, 100, 64, 64, 64, T, 0.02, seed=71)
    gamma = np.array([64, 1, 63, 0, 40], np.int32)
    li, g, cu_q, cu_d = case(cfg, gamma=gamma, T=T, sigma=0.02)
    gpu, ref, _, _ = check_accept(li, T, g, cu_q, cu_d, cfg.gamma_max)
    assert ref.n_accepted.max() >= 8


def test_full_size_c5_sampled_sequences():
    """The largest configuration at full size, launched as the benchmark launches it (batch 128,
    gamma 16 for every sequence, fixed row slabs): 12 sampled sequences against the oracle."""
    cfg = synth.scaled(synth.CONFIGS["c5"], gamma_lo=16, gamma_hi=16)
    li, g, cu_q, cu_d = case(cfg, padded=True)
    gpu = run_accept_gpu(li, cfg.temperature, g, cu_q, cu_d, cfg.gamma_max)
    assert gpu.status == 0
    pick = np.sort(np.random.default_rng(5).choice(cfg.batch, 12, replace=False))
    q_rows = np.concatenate([np.arange(cu_q[b], cu_q[b + 1]) for b in pick])
    d_rows = np.concatenate([np.arange(cu_d[b], cu_d[b + 1]) for b in pick])
    sub = synth.LogitInputs(li.target_logits[q_rows], li.draft_logits[d_rows], li.draft_tokens[d_rows],
                            li.u_accept[d_rows], li.u_sample[pick])
    sub_q, sub_d = synth.padded_offsets(len(pick), cfg.gamma_max)
    from tests.harness import AcceptOut
    gpu_sub = AcceptOut(gpu.n_accepted[pick], gpu.out_tokens[pick], gpu.ratio[d_rows], gpu.logZ_p[q_rows],
                        gpu.logZ_q[d_rows], 0, 0)
    ref, _, _ = compare_accept(gpu_sub, sub, cfg.temperature, g[pick], sub_q, sub_d, cfg.gamma_max)
    seen = np.isfinite(ref.logZ_p)            # rows the oracle evaluated (up to the first rejection)
    assert seen.any() and np.abs(np.expm1(gpu_sub.logZ_p[seen] - ref.logZ_p[seen])).max() <= 1e-5
    # properties that hold at any size: counts in range, accepted tokens are the drafts, one
    # token follows them and padding after it
    assert ((gpu.n_accepted >= 0) & (gpu.n_accepted <= g)).all()
    for b in range(cfg.batch):
        n = gpu.n_accepted[b]
        assert np.array_equal(gpu.out_tokens[b, :n], li.draft_tokens[cu_d[b]:cu_d[b] + n])
        assert 0 <= gpu.out_tokens[b, n] < cfg.vocab and (gpu.out_tokens[b, n + 1:] == -1).all()


@pytest.mark.parametrize("V", [1, 2, 3, 5, 127, 129, 1001, 4099])
def test_small_and_odd_vocabularies(V):
    # V < one warp segment, V % 4 != 0 (scalar loads, unaligned rows), ragged tails
    cfg = synth.VerifyConfig("odd", 9, 1, 1, 64, V, 32, 32, 0, 5, 5, 0.9, 0.7, seed=900 + V)
    for step in range(3):
        li, g, cu_q, cu_d = case(cfg, step=step)
        check_accept(li, cfg.temperature, g, cu_q, cu_d, cfg.gamma_max)


def test_row_stride_larger_than_vocab():
    cfg = synth.VerifyConfig("stride", 4, 1, 1, 64, 1000, 32, 32, 1, 4, 4, 1.0, 0.5, seed=77)
    li, g, cu_q, cu_d = case(cfg)
    n_q, n_d, V, S = int(cu_q[-1]), int(cu_d[-1]), 1000, 1024
    tl = torch.full((n_q, S), 50.0, dtype=torch.float32, device=DEV)      # poison in the padding
    dl = torch.full((n_d, S), 50.0, dtype=torch.float32, device=DEV)
    tl[:, :V] = dev(li.target_logits)
    dl[:, :V] = dev(li.draft_logits)
    n_acc = torch.zeros(4, dtype=torch.int32, device=DEV)
    out = torch.zeros((4, 5), dtype=torch.int32, device=DEV)
    ws = torch.empty(sv.spec_accept_sample_workspace_bytes(4, 4, S), dtype=torch.uint8, device=DEV)
    # padded buffers go in whole; the true vocabulary is set by hand
    p = sv.accept_params(tl, dl, dev(li.draft_tokens), dev(li.u_accept), dev(li.u_sample), 1.0, dev(g),
                         dev(cu_q), dev(cu_d), 4, n_acc, out)
    p.vocab = V
    st = sv.load().spec_accept_sample(C.byref(p), ws.data_ptr(), ws.numel(), None)
    assert st == 0
    torch.cuda.synchronize()
    ref = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept,
                               li.u_sample, 1.0, g, cu_q, cu_d, 4)
    np.testing.assert_array_equal(n_acc.cpu().numpy(), ref.n_accepted)
    np.testing.assert_array_equal(out.cpu().numpy(), ref.out_tokens)


def test_mixed_temperatures_per_sequence():
    cfg = synth.VerifyConfig("mix", 12, 1, 1, 64, 5000, 32, 32, 0, 6, 6, 1.0, 0.6, seed=31)
    li, g, cu_q, cu_d = case(cfg)
    T = np.array([0.0, 1.0, 0.5, 0.0, 2.0, 1.0, 0.0, 0.7, 1.3, 0.0, 1.0, 0.25], np.float32)
    # greedy sequences: make most draft tokens the target argmax so that several are accepted
    for b in np.flatnonzero(T == 0):
        for i in range(g[b]):
            if i % 3 != 2:
                li.draft_tokens[cu_d[b] + i] = int(np.argmax(li.target_logits[cu_q[b] + i]))
    check_accept(li, 1.0, g, cu_q, cu_d, cfg.gamma_max, temperature_per_seq=T)


def test_greedy_ties_take_lowest_index():
    B, V, gmax = 8, 3000, 3
    rng = np.random.default_rng(5)
    gamma = np.full(B, gmax, np.int32)
    cu_q, cu_d = synth.prefix(gamma)
    tl = rng.integers(-2, 3, (cu_q[-1], V)).astype(np.float32)       # the maximum repeats many times
    dl = np.zeros((cu_d[-1], V), np.float32)
    first = np.array([int(np.flatnonzero(r == r.max())[0]) for r in tl], np.int32)
    x = np.concatenate([first[cu_q[b]:cu_q[b] + gmax] for b in range(B)])
    x[5] = (x[5] + 1) % V
    li = synth.LogitInputs(tl, dl, x, np.zeros(cu_d[-1], np.float32), np.zeros(B, np.float32))
    gpu, ref, _, _ = check_accept(li, 0.0, gamma, cu_q, cu_d, gmax)
    assert ref.n_accepted.tolist().count(gmax) == B - 1


def test_masked_vocabulary_and_disjoint_supports():
    # -inf logits: tokens that cannot occur; disjoint supports reject at once and resample from p
    V, B = 600, 64
    rng = np.random.default_rng(8)
    p = np.zeros(V); p[:300] = rng.dirichlet(np.ones(300))
    q = np.zeros(V); q[300:] = rng.dirichlet(np.ones(300))
    gamma = np.full(B, 2, np.int32)
    cu_q, cu_d = synth.prefix(gamma)
    tl = np.tile(logits_of(p), (cu_q[-1], 1))
    dl = np.tile(logits_of(q), (cu_d[-1], 1))
    x = draw_from(rng, q, cu_d[-1])
    li = synth.LogitInputs(tl, dl, x, rng.random(cu_d[-1], dtype=np.float32), rng.random(B, dtype=np.float32))
    gpu, ref, _, _ = check_accept(li, 1.0, gamma, cu_q, cu_d, 2)
    assert (gpu.n_accepted == 0).all() and (gpu.out_tokens[:, 0] < 300).all()


def test_identical_models_and_zero_residual():
    V, B = 777, 16
    rng = np.random.default_rng(9)
    gamma = np.full(B, 3, np.int32)
    cu_q, cu_d = synth.prefix(gamma)
    tl = (2 * rng.standard_normal((cu_q[-1], V))).astype(np.float32)
    dl = np.concatenate([tl[cu_q[b]:cu_q[b] + 3] for b in range(B)])
    x = rng.integers(0, V, cu_d[-1]).astype(np.int32)
    li = synth.LogitInputs(tl, dl, x, rng.random(cu_d[-1], dtype=np.float32), rng.random(B, dtype=np.float32))
    gpu, ref, _, _ = check_accept(li, 1.0, gamma, cu_q, cu_d, 3)
    assert (gpu.n_accepted == 3).all()
    assert np.nanmax(np.abs(gpu.ratio - 1.0)) < 1e-6


def test_emitted_distribution_on_device():
    # the chi-square exactness pin, run through the CUDA kernels: V = 8, gamma = 2
    V, gamma, N = 8, 2, 200_000
    rng = np.random.default_rng(21)
    p_rows = [rng.dirichlet(np.ones(V)) for _ in range(gamma + 1)]
    q_rows = [rng.dirichlet(np.ones(V)) for _ in range(gamma)]
    tl = np.tile(np.stack([logits_of(p) for p in p_rows]), (N, 1))
    dl = np.tile(np.stack([logits_of(q) for q in q_rows]), (N, 1))
    x = np.stack([draw_from(rng, q, N) for q in q_rows], 1).reshape(-1)
    g = np.full(N, gamma, np.int32)
    cu_q, cu_d = synth.prefix(g)
    li = synth.LogitInputs(tl, dl, x, rng.random(N * gamma, dtype=np.float32), rng.random(N, dtype=np.float32))
    gpu = run_accept_gpu(li, 1.0, g, cu_q, cu_d, gamma)
    for j in range(gamma + 1):
        sel = gpu.n_accepted >= j
        assert chi2_p(gpu.out_tokens[sel, j], p_rows[j]) > 1e-3
    compare_accept(gpu, li, 1.0, g, cu_q, cu_d, gamma)


def test_device_status_bits():
    cfg = synth.VerifyConfig("bad", 4, 1, 1, 64, 512, 32, 32, 2, 2, 2, 1.0, 0.5, seed=5)
    li, g, cu_q, cu_d = case(cfg)
    li.draft_tokens[0] = 9999                     # outside the vocabulary: rejected + status bit
    li.target_logits[cu_q[2] + 0, 7] = np.nan     # NaN logit: sequence 2 emits -1 + status bit
    gpu = run_accept_gpu(li, 1.0, g, cu_q, cu_d, 2)
    assert gpu.status & sv.SV_DEV_BAD_TOKEN and gpu.status & sv.SV_DEV_NONFINITE
    assert gpu.n_accepted[0] == 0 and gpu.out_tokens[0, 0] >= 0
    assert gpu.n_accepted[2] == 0 and (gpu.out_tokens[2] == -1).all()
    # sequences 1 and 3 are untouched by their neighbours' faults
    ref = oracle.accept_sample(li.target_logits, li.draft_logits, np.clip(li.draft_tokens, 0, 511),
                               li.u_accept, li.u_sample, 1.0, g, cu_q, cu_d, 2)
    for b in (1, 3):
        assert gpu.n_accepted[b] == ref.n_accepted[b]
        np.testing.assert_array_equal(gpu.out_tokens[b], ref.out_tokens[b])


@pytest.mark.parametrize("name", ["c1", "c3", "c4"])
def test_bf16_logits(name):
    """Logits stored as bf16: the device widens them exactly, so the result is the oracle's on the widened values
    (the same bit-exact comparison as for float32 logits), for the vectorised and the element-wise loads."""
    from tests.harness import bf16_rounded
    cfg = synth.CONFIGS[name]
    if name == "c4":
        cfg = synth.scaled(cfg, batch=8)
    li, g, cu_q, cu_d = case(cfg, padded=(name == "c4"))
    check_accept(bf16_rounded(li), cfg.temperature, g, cu_q, cu_d, cfg.gamma_max, bf16=True)
    check_accept(bf16_rounded(synth.LogitInputs(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept,
                                                li.u_sample)), 0.0, g, cu_q, cu_d, cfg.gamma_max, bf16=True)


@pytest.mark.parametrize("V", [1, 5, 8, 1000, 4099])
def test_bf16_logits_small_and_odd_vocabularies(V):
    from tests.harness import bf16_rounded
    cfg = synth.VerifyConfig("odd16", 3, 1, 1, 64, V, 32, 32, 0, 3, 3, 0.9, 0.7, seed=91 + V)
    li, g, cu_q, cu_d = case(cfg)
    check_accept(bf16_rounded(li), cfg.temperature, g, cu_q, cu_d, cfg.gamma_max, bf16=True)


@pytest.mark.parametrize("T", [0.05, 0.2, 4.0])
def test_low_and_high_temperatures_keep_the_ratio_bound(T):
    """The device forms ln Z from float32 exponentials of x * log2(e)/T - ref.  At a small temperature the products
    are large (|x| / T up to ~200 here) and the reference nearly cancels them: the split of log2(e)/T into two
    floats and the fused multiply-adds must keep the ratio within 1e-6 of the float64 one (check_accept asserts
    it for every evaluated position), or decisions outside the flagged window would flip."""
    cfg = synth.VerifyConfig("temp", 12, 1, 1, 64, 32000, 32, 32, 1, 6, 6, T, 0.6, seed=1000 + int(T * 100))
    li, g, cu_q, cu_d = case(cfg)
    gpu, ref, n_pos, n_tok = check_accept(li, T, g, cu_q, cu_d, cfg.gamma_max)
    assert np.isfinite(ref.ratio).sum() >= 12


def test_greedy_rows_without_an_argmax_set_the_status_bit():
    """T = 0: a target row that is all -inf, or holds a NaN or +inf, has no argmax.  The header promises
    SV_DEV_NONFINITE, no accepted drafts and -1 tokens for such a sequence, and nothing else changes."""
    cfg = synth.VerifyConfig("bad0", 5, 1, 1, 64, 4100, 32, 32, 3, 3, 3, 0.0, 0.5, seed=11)
    li, g, cu_q, cu_d = case(cfg)
    li.target_logits[cu_q[0] + 0, :] = -np.inf            # sequence 0: the first row is all -inf
    li.target_logits[cu_q[1] + 2, 4097] = np.nan          # sequence 1: a NaN in its third row (last slice)
    li.target_logits[cu_q[3] + 1, 17] = np.inf            # sequence 3: +inf in its second row
    li.draft_tokens[cu_d[1]:cu_d[1] + 2] = np.argmax(li.target_logits[cu_q[1]:cu_q[1] + 2], axis=1)   # two accepted first
    li.draft_tokens[cu_d[3]] = np.argmax(li.target_logits[cu_q[3]])                                     # one accepted first
    gpu = run_accept_gpu(li, 0.0, g, cu_q, cu_d, 3)
    assert gpu.status & sv.SV_DEV_NONFINITE
    for b in (0, 1, 3):
        assert gpu.n_accepted[b] == 0 and (gpu.out_tokens[b] == -1).all(), (b, gpu.out_tokens[b])
    clean = li.target_logits.copy()
    for b in (0, 1, 3):
        clean[cu_q[b]:cu_q[b + 1]] = 0.0
    ref = oracle.accept_sample(clean, li.draft_logits, li.draft_tokens, li.u_accept, li.u_sample, 0.0, g, cu_q,
                               cu_d, 3)
    for b in (2, 4):
        assert gpu.n_accepted[b] == ref.n_accepted[b]
        np.testing.assert_array_equal(gpu.out_tokens[b], ref.out_tokens[b])


def test_host_errors():
    t = torch.zeros((4, 100), dtype=torch.float32, device=DEV)
    i32 = torch.zeros(8, dtype=torch.int32, device=DEV)
    ws = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(sv.SpecVerifyError) as e:
        sv.spec_accept_sample(t, t, i32, t[0], t[0], 1.0, i32[:2], i32[:3], i32[:3], 1, i32[:2],
                              i32[:4].reshape(2, 2), ws)
    assert e.value.status == sv.SV_EWORKSPACE
