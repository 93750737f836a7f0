"""spec_kv_append on the GPU against the oracle: the pools after the call are compared bit for bit,
whole, so that a write to a wrong place is caught as well as a missing one."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import DEV, bits_of, dev, dev_bf16, run_attn_oracle, AttnCase, workspace

pytestmark = pytest.mark.gpu


def new_rows(cfg, n_rows, tensor):
    rng = np.random.default_rng([cfg.seed, tensor])
    return synth.bf16_bits(rng.standard_normal((n_rows, cfg.hkv, cfg.head_dim)).astype(np.float32))


def append_gpu(kv, k_new, v_new, seq_len, gamma, cu_q, gamma_max, pools=None):
    k, v = pools if pools is not None else (dev_bf16(kv.k_pool), dev_bf16(kv.v_pool))
    pool = sv.spec_kv_pool_register(k, v)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sv.spec_kv_append(dev_bf16(k_new), dev_bf16(v_new), pool, dev(kv.block_table), dev(seq_len), dev(gamma),
                      dev(cu_q), gamma_max, device_status=status)
    torch.cuda.synchronize()
    return k, v, pool, int(status.item())


def check_case(cfg, seq_len=None, gamma=None, padded=False):
    sl, g = synth.draw_lengths(cfg)
    if seq_len is not None:
        sl = np.asarray(seq_len, np.int32)
    if gamma is not None:
        g = np.asarray(gamma, np.int32)
    cu_q, _ = synth.padded_offsets(cfg.batch, cfg.gamma_max) if padded else synth.prefix(g)
    kv = synth.make_kv(cfg, sl)
    n = int(cu_q[-1])
    k_new, v_new = new_rows(cfg, n, 1), new_rows(cfg, n, 2)
    k, v, _, status = append_gpu(kv, k_new, v_new, sl, g, cu_q, cfg.gamma_max)
    assert status == 0
    k_ref, v_ref = oracle.kv_append(k_new, v_new, kv.k_pool, kv.v_pool, kv.strides, kv.block_table, sl, g, cu_q,
                                    cfg.page_size)
    np.testing.assert_array_equal(bits_of(k), k_ref)
    np.testing.assert_array_equal(bits_of(v), v_ref)
    assert (k_ref != kv.k_pool).any()
    return kv, k_new, v_new, sl, g, cu_q


@pytest.mark.parametrize("name,batch", [("c1", None), ("c2", None), ("c3", None), ("c4", 6), ("c5", 9)])
def test_config_shapes(name, batch):
    cfg = synth.CONFIGS[name]
    if batch:
        cfg = synth.scaled(cfg, batch=batch)
    check_case(cfg)


def test_page_boundaries_and_degenerate_blocks():
    cfg = synth.VerifyConfig("edge", 8, 8, 2, 128, 100, 1, 200, 0, 16, 16, 1.0, 1.0, seed=61)
    # blocks that end on, start on and straddle a page boundary; a sequence that is only its block
    # (R = L); gamma 0; one token in all
    gamma = np.array([3, 15, 16, 0, 16, 0, 7, 2], np.int32)
    seq_len = np.array([16, 32, 40, 1, 17, 33, 8, 19], np.int32)
    check_case(cfg, seq_len, gamma)
    check_case(cfg, seq_len, gamma, padded=True)


def test_slot_major_pool_layout():
    cfg = synth.VerifyConfig("slot", 4, 8, 4, 64, 100, 20, 300, 1, 6, 6, 1.0, 1.0, seed=62)
    sl, g = synth.draw_lengths(cfg)
    cu_q, _ = synth.prefix(g)
    kv = synth.make_kv(cfg, sl)
    n = int(cu_q[-1])
    k_new, v_new = new_rows(cfg, n, 1), new_rows(cfg, n, 2)
    # the same logical pool stored [page, slot, head, dim]
    k_sm = dev_bf16(np.ascontiguousarray(kv.k_pool.transpose(0, 2, 1, 3)))
    v_sm = dev_bf16(np.ascontiguousarray(kv.v_pool.transpose(0, 2, 1, 3)))
    k, v, _, status = append_gpu(kv, k_new, v_new, sl, g, cu_q, cfg.gamma_max,
                                 pools=(k_sm.permute(0, 2, 1, 3), v_sm.permute(0, 2, 1, 3)))
    assert status == 0
    k_ref, v_ref = oracle.kv_append(k_new, v_new, kv.k_pool, kv.v_pool, kv.strides, kv.block_table, sl, g, cu_q,
                                    cfg.page_size)
    np.testing.assert_array_equal(bits_of(k_sm).transpose(0, 2, 1, 3), k_ref)
    np.testing.assert_array_equal(bits_of(v_sm).transpose(0, 2, 1, 3), v_ref)


def test_append_then_attention_follows_the_oracle_chain():
    cfg = synth.VerifyConfig("chain", 5, 16, 4, 128, 100, 30, 700, 2, 9, 9, 1.0, 1.0, q_scale=3.0, seed=63)
    kv, k_new, v_new, sl, g, cu_q = check_case(cfg)
    k, v, pool, _ = append_gpu(kv, k_new, v_new, sl, g, cu_q, cfg.gamma_max)
    q_bits = synth.make_q(cfg, int(cu_q[-1]))
    q = dev_bf16(q_bits)
    o = torch.zeros_like(q)
    max_len = int(sl.max())
    ws = workspace(sv.spec_verify_attn_workspace_bytes(cfg.batch, cfg.gamma_max, cfg.hq, cfg.hkv, cfg.head_dim, max_len))
    sv.spec_verify_attn(q, o, pool, dev(kv.block_table), dev(sl), dev(g), dev(cu_q), cfg.gamma_max, max_len, ws)
    torch.cuda.synchronize()
    k_ref, v_ref = oracle.kv_append(k_new, v_new, kv.k_pool, kv.v_pool, kv.strides, kv.block_table, sl, g, cu_q,
                                    cfg.page_size)
    kv2 = synth.KVState(k_ref, v_ref, kv.block_table, kv.strides)
    o_ref, _ = run_attn_oracle(AttnCase(cfg, sl, g, cu_q, kv2, q_bits))
    o_gpu = synth.bf16_to_f32(bits_of(o)).astype(np.float64)
    assert np.abs(o_gpu - o_ref).max() <= 2e-2
    # the new rows matter: attention over the cache before the append differs
    o_old, _ = run_attn_oracle(AttnCase(cfg, sl, g, cu_q, kv, q_bits))
    assert np.abs(o_old - o_ref).max() > 0.1


def test_device_detected_conditions():
    cfg = synth.VerifyConfig("bad", 4, 8, 2, 128, 100, 40, 100, 2, 4, 4, 1.0, 1.0, seed=64)
    sl, g = synth.draw_lengths(cfg)
    cu_q, _ = synth.padded_offsets(cfg.batch, cfg.gamma_max)
    kv = synth.make_kv(cfg, sl)
    n = int(cu_q[-1])
    k_new, v_new = new_rows(cfg, n, 1), new_rows(cfg, n, 2)
    # sequence 1: a page id out of range at the block's last position; sequence 2: shorter than its block;
    # sequence 3: gamma above the bound (clamped to gamma_max)
    bt = kv.block_table.copy()
    bt[1, (sl[1] - 1) // 16] = 10 ** 6
    sl_bad = sl.copy()
    sl_bad[2] = g[2]
    g_bad = g.copy()
    g_bad[3] = cfg.gamma_max + 5
    kv_bad = synth.KVState(kv.k_pool, kv.v_pool, bt, kv.strides)
    k, v, _, status = append_gpu(kv_bad, k_new, v_new, sl_bad, g_bad, cu_q, cfg.gamma_max)
    assert status == sv.SV_DEV_BAD_PAGE | sv.SV_DEV_BAD_LEN | sv.SV_DEV_BAD_GAMMA
    # expected: the oracle on the inputs as the device repaired or skipped them
    g_fix = g_bad.copy()
    g_fix[3] = cfg.gamma_max
    k_ref, v_ref = kv.k_pool, kv.v_pool
    for b in (0, 3):
        one = lambda a: np.asarray(a[b:b + 1])
        k_ref, v_ref = oracle.kv_append(k_new[cu_q[b]:cu_q[b + 1]], v_new[cu_q[b]:cu_q[b + 1]], k_ref, v_ref, kv.strides,
                                        one(kv.block_table), one(sl_bad), one(g_fix), [0, cfg.gamma_max + 1], cfg.page_size)
    # sequence 1: the positions in its last page are skipped, those in the page before are written
    R1 = g[1] + 1
    first = sl[1] - R1
    keep = [i for i in range(R1) if (first + i) // 16 != (sl[1] - 1) // 16]
    for i in keep:
        pos = first + i
        k_ref[kv.block_table[1, pos // 16], :, pos % 16] = k_new[cu_q[1] + i]
        v_ref[kv.block_table[1, pos // 16], :, pos % 16] = v_new[cu_q[1] + i]
    np.testing.assert_array_equal(bits_of(k), k_ref)
    np.testing.assert_array_equal(bits_of(v), v_ref)


def test_host_errors():
    cfg = synth.VerifyConfig("host", 2, 8, 2, 128, 100, 40, 60, 1, 2, 2, 1.0, 1.0, seed=65)
    sl, g = synth.draw_lengths(cfg)
    cu_q, _ = synth.prefix(g)
    kv = synth.make_kv(cfg, sl)
    pool = sv.spec_kv_pool_register(dev_bf16(kv.k_pool), dev_bf16(kv.v_pool))
    n = int(cu_q[-1])
    kn = dev_bf16(new_rows(cfg, n, 1))
    with pytest.raises(ValueError):
        sv.spec_kv_append(kn[:, :1], kn[:, :1], pool, dev(kv.block_table), dev(sl), dev(g), dev(cu_q), cfg.gamma_max)
    import ctypes as C
    p = sv.kv_append_params(kn, kn, pool, dev(kv.block_table), dev(sl), dev(g), dev(cu_q), cfg.gamma_max)
    p.k_new = kn.data_ptr() + 2
    assert sv.load().spec_kv_append(C.byref(p), None) == sv.SV_EALIGN
    p.k_new = None
    assert sv.load().spec_kv_append(C.byref(p), None) == sv.SV_EINVAL
    assert sv.load().spec_kv_append(None, None) == sv.SV_EINVAL


def test_full_size_c5():
    # the benchmark's configuration: every sequence at gamma 16, whole pools compared on the device
    cfg = synth.CONFIGS["c5"]
    sl, _ = synth.draw_lengths(cfg)
    g = np.full(cfg.batch, cfg.gamma_max, np.int32)
    cu_q, _ = synth.padded_offsets(cfg.batch, cfg.gamma_max)
    kv = synth.make_kv(cfg, sl)
    n = int(cu_q[-1])
    k_new, v_new = new_rows(cfg, n, 1), new_rows(cfg, n, 2)
    k, v, _, status = append_gpu(kv, k_new, v_new, sl, g, cu_q, cfg.gamma_max)
    assert status == 0
    k_ref, v_ref = oracle.kv_append(k_new, v_new, kv.k_pool, kv.v_pool, kv.strides, kv.block_table, sl, g, cu_q,
                                    cfg.page_size)
    assert torch.equal(k.view(torch.int16), dev_bf16(k_ref).view(torch.int16))
    assert torch.equal(v.view(torch.int16), dev_bf16(v_ref).view(torch.int16))
    changed = int((k.view(torch.int16) != dev_bf16(kv.k_pool).view(torch.int16)).sum().item())
    assert 0.99 * n * cfg.hkv * cfg.head_dim <= changed <= n * cfg.hkv * cfg.head_dim
