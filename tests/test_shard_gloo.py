"""The N > 1 path on CPU: batch partitioning, and two `gloo` ranks that each run the
verify step on their own shard (with the oracle standing in for the GPU) and must
reproduce the whole-batch result exactly -- sequences are independent, so sharding may
not change a single bit."""
import os
import socket
import tempfile

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2504_00030_b200 import shard, synth


def test_shard_bounds_cover_and_balance():
    for n in (0, 1, 2, 7, 128, 129):
        for world in (1, 2, 3, 8):
            b = shard.shard_bounds(n, world)
            assert b[0] == 0 and b[-1] == n and len(b) == world + 1
            sizes = np.diff(b)
            assert (sizes >= 0).all() and sizes.max() - sizes.min() <= 1
            assert (np.diff(sizes) <= 0).all()          # the larger shards come first
    with pytest.raises(ValueError):
        shard.shard_bounds(4, 0)


def test_balanced_bounds_by_context_length():
    rng = np.random.default_rng(5)
    cost = rng.integers(512, 16385, size=128)
    for world in (1, 2, 4, 8):
        b = shard.balanced_bounds(cost, world)
        assert b[0] == 0 and b[-1] == 128 and (np.diff(b) >= 0).all()
        per = np.add.reduceat(cost, b[:-1])[:world] if world > 1 else np.array([cost.sum()])
        # a contiguous cut can miss the ideal share by at most one sequence's cost
        assert np.abs(per - cost.sum() / world).max() <= cost.max()
    # degenerate inputs: empty batch, all-zero costs
    assert shard.balanced_bounds(np.zeros(0), 4).tolist() == [0, 0, 0, 0, 0]
    assert shard.balanced_bounds(np.zeros(3), 2)[-1] == 3


def test_local_batch_rebases_offsets():
    gamma = np.array([3, 0, 5, 2, 4], np.int32)
    seq_len = np.array([40, 17, 90, 33, 64], np.int32)
    cu_q, cu_d = synth.prefix(gamma)
    b = shard.shard_bounds(5, 2)                        # 3 + 2
    l0 = shard.local_batch(b, 0, seq_len, gamma, cu_q, cu_d)
    l1 = shard.local_batch(b, 1, seq_len, gamma, cu_q, cu_d)
    assert (l0.first, l0.count, l1.first, l1.count) == (0, 3, 3, 2)
    assert l0.cu_q.tolist() == [0, 4, 5, 11] and l0.cu_d.tolist() == [0, 3, 3, 8]
    assert l1.cu_q.tolist() == [0, 3, 8] and l1.cu_d.tolist() == [0, 2, 6]
    assert (l0.q_rows, l1.q_rows) == (slice(0, 11), slice(11, 19))
    assert (l0.d_rows, l1.d_rows) == (slice(0, 8), slice(8, 14))
    # padded slabs stay padded
    pq, pd = synth.padded_offsets(5, 6)
    p1 = shard.local_batch(b, 1, seq_len, gamma, pq, pd)
    assert p1.cu_q.tolist() == [0, 7, 14] and p1.cu_d.tolist() == [0, 6, 12]
    assert p1.q_rows == slice(21, 35)


CFG = synth.scaled(synth.CONFIGS["c3"], batch=5, hq=4, hkv=2, head_dim=32, vocab=257, ctx_lo=20, ctx_hi=90,
                   gamma_lo=0, gamma_hi=5, gamma_max=5, seed=77)
GT = dict(eta=0.5, delta=2.0, gamma_min=1)


def whole_batch():
    seq_len, gamma = synth.draw_lengths(CFG)
    cu_q, cu_d = synth.prefix(gamma)
    kv = synth.make_kv(CFG, seq_len)
    q = synth.make_q(CFG, int(cu_q[-1]))
    li = synth.make_logits(CFG, gamma, cu_q, cu_d)
    return seq_len, gamma, cu_q, cu_d, kv, q, li


def verify_step(seq_len, gamma, cu_q, cu_d, kv, block_table, q, tl, dl, x, ua, us):
    scale = float(np.float32(CFG.head_dim ** -0.5))
    o, _ = oracle.verify_attn(q, kv.k_pool, kv.v_pool, kv.strides, block_table, seq_len, gamma, cu_q, CFG.hq,
                              CFG.hkv, CFG.page_size, scale)
    res = oracle.accept_sample(tl, dl, x, ua, us, CFG.temperature, gamma, cu_q, cu_d, CFG.gamma_max)
    gbar, g, sl, _, _ = oracle.gamma_tune_update(res.n_accepted, gamma.astype(np.float64), gamma, seq_len,
                                                 GT["eta"], GT["delta"], GT["gamma_min"], CFG.gamma_max,
                                                 oracle.MODE_GT_PROPOSED, False)
    return o, res.n_accepted, res.out_tokens, gbar, g, sl


def _rank_main(rank, world, port, outdir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seq_len, gamma, cu_q, cu_d, kv, q, li = whole_batch()
        bounds = shard.balanced_bounds(seq_len, world) if world == 2 else shard.shard_bounds(CFG.batch, world)
        lb = shard.local_batch(bounds, rank, seq_len, gamma, cu_q, cu_d)
        sl_ = slice(lb.first, lb.first + lb.count)
        o, n_acc, toks, gbar, g, sl = verify_step(
            lb.seq_len, lb.gamma, lb.cu_q, lb.cu_d, kv, kv.block_table[sl_], q[lb.q_rows],
            li.target_logits[lb.q_rows], li.draft_logits[lb.d_rows], li.draft_tokens[lb.d_rows],
            li.u_accept[lb.d_rows], li.u_sample[sl_])
        gathered = {
            "n_acc": shard.gather_sequences(torch.from_numpy(n_acc), bounds),
            "toks": shard.gather_sequences(torch.from_numpy(toks), bounds),
            "gbar": shard.gather_sequences(torch.from_numpy(gbar), bounds),
            "g": shard.gather_sequences(torch.from_numpy(g), bounds),
            "sl": shard.gather_sequences(torch.from_numpy(sl), bounds),
        }
        # attention rows are per row, not per sequence: gather through row boundaries
        row_bounds = np.asarray(cu_q, np.int64)[bounds]
        gathered["o"] = shard.gather_sequences(torch.from_numpy(o), row_bounds)
        # timing reduction: rank r pretends its step took 1 + r ms and verified these tokens
        (ms,), tokens = shard.reduce_timing([1.0 + rank], int((n_acc + 1).sum()))
        gathered["ms"] = torch.tensor([ms])
        gathered["tokens"] = torch.tensor([tokens])
        torch.save(gathered, os.path.join(outdir, f"rank{rank}.pt"))
    finally:
        dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.timeout(300)
def test_two_gloo_ranks_reproduce_the_whole_batch():
    oracle.build()
    world = 2
    with tempfile.TemporaryDirectory() as outdir:
        mp.spawn(_rank_main, args=(world, _free_port(), outdir), nprocs=world, join=True)
        got = [torch.load(os.path.join(outdir, f"rank{r}.pt")) for r in range(world)]
    seq_len, gamma, cu_q, cu_d, kv, q, li = whole_batch()
    o, n_acc, toks, gbar, g, sl = verify_step(seq_len, gamma, cu_q, cu_d, kv, kv.block_table, q, li.target_logits,
                                              li.draft_logits, li.draft_tokens, li.u_accept, li.u_sample)
    for r in range(world):
        assert np.array_equal(got[r]["n_acc"].numpy(), n_acc)
        assert np.array_equal(got[r]["toks"].numpy(), toks)
        assert np.array_equal(got[r]["g"].numpy(), g)
        assert np.array_equal(got[r]["sl"].numpy(), sl)
        assert np.array_equal(got[r]["gbar"].numpy(), gbar)          # bit-identical float64
        assert np.array_equal(got[r]["o"].numpy(), o)
        assert got[r]["ms"].item() == 2.0                            # max over ranks
        assert got[r]["tokens"].item() == int((n_acc + 1).sum())     # sum over ranks


def test_reduce_timing_without_a_process_group():
    ms, tokens = shard.reduce_timing([1.5, 2.5], 7)
    assert ms == [1.5, 2.5] and tokens == 7
    t = torch.arange(6).reshape(3, 2)
    assert shard.gather_sequences(t, np.array([0, 3])) is t
