"""spec_verify_attn on the GPU against the oracle: |o - o_ref| <= 2e-2, softmax sums to 1e-5."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import (ATTN_ATOL, DEV, AttnCase, bits_of, check_attn, dev, dev_bf16,
                           make_attn_case, run_attn_gpu, run_attn_oracle, used_rows, workspace)

pytestmark = pytest.mark.gpu


def test_config_c1_tiny():
    check_attn(make_attn_case(synth.CONFIGS["c1"]))


def test_config_c2_shape():
    cfg = synth.CONFIGS["c2"]
    for gam in (1, 8):
        check_attn(make_attn_case(cfg, gamma=[gam]))


@pytest.mark.parametrize("q_scale", [1.0, 6.0])
def test_config_c3_shape_reduced_batch(q_scale):
    # q_scale 6 makes the softmax peaky so that |o| is O(1) and the 2e-2 bound bites
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=4, ctx_lo=900, ctx_hi=3000, q_scale=q_scale)
    check_attn(make_attn_case(cfg))


@pytest.mark.parametrize("q_scale", [1.0, 6.0])
def test_config_c3_at_its_stated_size(q_scale):
    """Llama-3.1-8B shape as the workload states it: batch 16, 32q/8kv heads, contexts 1024..8192,
    gamma 2..10; every output row against the oracle (plain inputs, and peaky ones so the bound bites)."""
    check_attn(make_attn_case(synth.scaled(synth.CONFIGS["c3"], q_scale=q_scale)))


def test_config_c4_shape_reduced():
    cfg = synth.scaled(synth.CONFIGS["c4"], batch=3, hq=8, hkv=8, ctx_lo=4096, ctx_hi=4096, q_scale=4.0)
    check_attn(make_attn_case(cfg, padded=True))


def test_config_c5_shape_reduced_batch():
    # 8 query heads per kv head x 17 rows = 136 rows per (sequence, kv head)
    cfg = synth.scaled(synth.CONFIGS["c5"], batch=3, hq=16, hkv=2, ctx_lo=300, ctx_hi=2500, q_scale=5.0)
    check_attn(make_attn_case(cfg))


@pytest.mark.parametrize("D,hq,hkv", [(64, 4, 4), (128, 8, 2), (128, 4, 1)])
def test_short_and_edge_lengths(D, hq, hkv):
    # L around page and tile boundaries, block == whole context, gamma == 0
    cfg = synth.VerifyConfig("edge", 12, hq, hkv, D, 100, 1, 1, 0, 0, 16, 1.0, 1.0, q_scale=4.0, seed=41)
    seq_len = np.array([1, 2, 15, 16, 17, 31, 127, 128, 129, 255, 257, 17], np.int32)
    gamma = np.array([0, 1, 3, 15, 16, 0, 7, 2, 16, 5, 1, 16], np.int32)
    check_attn(make_attn_case(cfg, seq_len, gamma))


def test_ragged_gqa_many_sequences():
    cfg = synth.VerifyConfig("ragged", 37, 12, 4, 128, 100, 1, 1500, 0, 12, 12, 1.0, 1.0, q_scale=3.0,
                             seed=43)
    check_attn(make_attn_case(cfg))


def test_many_short_sequences():
    # far more (sequence, kv head) pairs than thread blocks, one tile each: every block's share is a
    # run of whole pairs, and the schedule's scans run over a batch of 1500
    cfg = synth.VerifyConfig("short", 1500, 8, 2, 128, 100, 1, 60, 0, 4, 4, 1.0, 1.0, q_scale=3.0, seed=52)
    check_attn(make_attn_case(cfg))


def test_mixed_row_counts_around_128():
    # 8 query heads per kv head, gamma from 0 to 16: pairs with 8 .. 136 rows in one launch,
    # so pairs that need the second row group alternate with pairs that do not
    cfg = synth.VerifyConfig("mixed", 20, 16, 2, 128, 100, 100, 1800, 0, 16, 16, 1.0, 1.0, q_scale=3.0,
                             seed=50)
    gamma = np.array([16, 15, 16, 0, 7, 16, 16, 14, 15, 16, 1, 16, 15, 15, 16, 3, 16, 16, 15, 2], np.int32)
    check_attn(make_attn_case(cfg, gamma=gamma))
    check_attn(make_attn_case(cfg, gamma=np.full(20, 15, np.int32)))


def test_more_than_144_rows_per_pair():
    # 16 query heads per kv head x up to 13 positions = 208 rows: the kernel with two 128-row groups
    cfg = synth.VerifyConfig("wide", 6, 32, 2, 128, 100, 200, 2600, 9, 12, 12, 1.0, 1.0, q_scale=3.0, seed=51)
    check_attn(make_attn_case(cfg))


def test_long_context_single_sequence():
    cfg = synth.VerifyConfig("long", 1, 8, 1, 128, 100, 16384, 16384, 16, 16, 16, 1.0, 1.0, q_scale=6.0,
                             seed=44)
    check_attn(make_attn_case(cfg))


def test_padded_row_layout():
    cfg = synth.VerifyConfig("pad", 5, 8, 2, 128, 100, 40, 900, 0, 6, 6, 1.0, 1.0, q_scale=3.0, seed=45)
    check_attn(make_attn_case(cfg, padded=True))


def test_physical_page_permutation():
    cfg = synth.VerifyConfig("perm", 3, 8, 2, 128, 100, 200, 700, 1, 5, 5, 1.0, 1.0, q_scale=3.0, seed=46)
    case = make_attn_case(cfg)
    o1, lse1, _ = run_attn_gpu(case)
    n_pages = case.kv.k_pool.shape[0]
    perm = np.random.default_rng(1).permutation(n_pages)
    k2, v2 = np.empty_like(case.kv.k_pool), np.empty_like(case.kv.v_pool)
    k2[perm], v2[perm] = case.kv.k_pool, case.kv.v_pool
    bt2 = np.where(case.kv.block_table >= 0, perm[np.maximum(case.kv.block_table, 0)], -1).astype(np.int32)
    case2 = AttnCase(cfg, case.seq_len, case.gamma, case.cu_q,
                     synth.KVState(k2, v2, bt2, case.kv.strides), case.q)
    o2, lse2, _ = run_attn_gpu(case2)
    rows = used_rows(case.gamma, case.cu_q)
    o_ref, _ = run_attn_oracle(case)
    assert np.abs(o1[rows] - o_ref[rows]).max() <= ATTN_ATOL
    assert np.abs(o2[rows] - o_ref[rows]).max() <= ATTN_ATOL
    np.testing.assert_array_equal(o1[rows], o2[rows])      # same arithmetic, only addresses moved


def test_pool_stored_page_slot_head_dim():
    cfg = synth.VerifyConfig("strided", 3, 8, 2, 128, 100, 100, 600, 1, 4, 4, 1.0, 1.0, q_scale=3.0, seed=47)
    case = make_attn_case(cfg)
    o_ref, lse_ref = run_attn_oracle(case)
    # store the pool as [page, slot, head, dim] and describe it through the strides
    k = dev_bf16(np.ascontiguousarray(case.kv.k_pool.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
    v = dev_bf16(np.ascontiguousarray(case.kv.v_pool.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
    pool = sv.spec_kv_pool_register(k, v)
    q = dev_bf16(case.q)
    o = torch.zeros_like(q)
    max_len = int(case.seq_len.max())
    ws = workspace(sv.spec_verify_attn_workspace_bytes(cfg.batch, cfg.gamma_max, cfg.hq, cfg.hkv, 128, max_len))
    sv.spec_verify_attn(q, o, pool, dev(case.kv.block_table), dev(case.seq_len), dev(case.gamma),
                        dev(case.cu_q), cfg.gamma_max, max_len, ws)
    torch.cuda.synchronize()
    rows = used_rows(case.gamma, case.cu_q)
    o_gpu = synth.bf16_to_f32(bits_of(o)).astype(np.float64)
    assert np.abs(o_gpu[rows] - o_ref[rows]).max() <= ATTN_ATOL


def test_bad_page_and_bad_length_set_status():
    cfg = synth.VerifyConfig("bad", 3, 4, 1, 128, 100, 100, 300, 2, 2, 2, 1.0, 1.0, seed=48)
    case = make_attn_case(cfg)
    o_ref, _ = run_attn_oracle(case)
    case.kv.block_table[1, 0] = 10_000_000           # page id outside the pool
    o, lse, status = run_attn_gpu(case)
    assert status & sv.SV_DEV_BAD_PAGE
    rows0 = np.arange(case.cu_q[0], case.cu_q[1])   # the other sequences are still right
    assert np.abs(o[rows0] - o_ref[rows0]).max() <= ATTN_ATOL
    case = make_attn_case(cfg)
    case.seq_len[2] = 1                              # shorter than its own draft block
    o, lse, status = run_attn_gpu(case)
    assert status & sv.SV_DEV_BAD_LEN


def test_host_errors():
    cfg = synth.VerifyConfig("err", 2, 4, 1, 128, 100, 100, 300, 2, 2, 2, 1.0, 1.0, seed=49)
    case = make_attn_case(cfg)
    k, v = dev_bf16(case.kv.k_pool), dev_bf16(case.kv.v_pool)
    pool = sv.spec_kv_pool_register(k, v)
    q = dev_bf16(case.q)
    o = torch.zeros_like(q)
    args = (dev(case.kv.block_table), dev(case.seq_len), dev(case.gamma), dev(case.cu_q))
    pool2 = sv.spec_kv_pool_register(k.repeat(1, 2, 1, 1), v.repeat(1, 2, 1, 1))
    with pytest.raises(sv.SpecVerifyError) as e:      # 3 query heads over 2 kv heads
        sv.spec_verify_attn(q[:, :3].contiguous(), o[:, :3].contiguous(), pool2, *args, 2, 300,
                            workspace(1 << 20))
    assert e.value.status == sv.SV_EUNSUPPORTED
    with pytest.raises(sv.SpecVerifyError) as e:      # block table narrower than max_seq_len needs
        sv.spec_verify_attn(q, o, pool, *args, 2, 100000, workspace(1 << 20))
    assert e.value.status == sv.SV_EINVAL


@pytest.mark.parametrize("name,q_scale", [("c5", 1.0), ("c4", 1.0), ("c4", 4.0)])
def test_full_size_sampled_rows(name, q_scale):
    """The two largest configurations at full size (c5: batch 128, 64q/8kv heads, contexts 512..16384, gamma 16;
    c4: batch 64, 40 heads, context 4096, gamma 1..12): 40 sampled (sequence, row, head) outputs each."""
    cfg = synth.scaled(synth.CONFIGS[name], q_scale=q_scale)
    case = make_attn_case(cfg)
    o_gpu, lse_gpu, status = run_attn_gpu(case)
    assert status == 0
    rng = np.random.default_rng(0)
    scale = float(np.float32(cfg.head_dim ** -0.5))
    worst = 0.0
    for _ in range(40):
        b = int(rng.integers(cfg.batch))
        i = int(rng.integers(case.gamma[b] + 1))
        h = int(rng.integers(cfg.hq))
        row = case.cu_q[b] + i
        n_keys = int(case.seq_len[b]) - (int(case.gamma[b]) + 1) + i + 1
        o_ref, lse_ref = oracle.attn_row(case.q[row, h], case.kv.k_pool, case.kv.v_pool, case.kv.strides,
                                         case.kv.block_table[b], cfg.page_size, h // cfg.group, n_keys, scale)
        worst = max(worst, np.abs(o_gpu[row, h] - o_ref).max())
        assert abs(np.expm1(lse_gpu[row, h] - lse_ref)) <= 1e-5
    assert worst <= ATTN_ATOL
    # property that holds at any size: every used output row is finite and inside the value range
    rows = used_rows(case.gamma, case.cu_q)
    assert np.isfinite(o_gpu[rows]).all() and np.abs(o_gpu[rows]).max() < 6.0
