"""spec_verify_attn_layers: the cache append and the verify attention of several layers' caches in one call
(one cache per layer behind one block table, KV caching of paper Section 5), against the oracle layer by layer."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth
from tests.harness import ATTN_ATOL, DEV, bits_of, dev, dev_bf16, used_rows, workspace

pytestmark = pytest.mark.gpu


def layer_inputs(cfg, n_layers, seq_len, n_q):
    """Distinct pools, queries and new rows per layer (the layers share lengths and block table)."""
    kvs, qs, news = [], [], []
    for l in range(n_layers):
        c = synth.scaled(cfg, seed=cfg.seed + 1000 * (l + 1))
        kv = synth.make_kv(c, seq_len, reserve_tokens=0)
        kvs.append(kv)
        qs.append(synth.make_q(c, n_q))
        n = n_q * cfg.hkv * cfg.head_dim
        news.append((synth.normal_bf16_bits(c.seed, 90, n).reshape(n_q, cfg.hkv, cfg.head_dim),
                     synth.normal_bf16_bits(c.seed, 91, n).reshape(n_q, cfg.hkv, cfg.head_dim)))
    return kvs, qs, news


@pytest.mark.parametrize("append", [True, False])
@pytest.mark.parametrize("name", ["gqa", "mha64"])
def test_layers_match_the_oracle_layer_by_layer(name, append):
    cfg = {"gqa": synth.VerifyConfig("layers", 5, 16, 4, 128, 100, 40, 900, 0, 7, 7, 1.0, 1.0, q_scale=3.0, seed=301),
           "mha64": synth.VerifyConfig("layers64", 3, 6, 6, 64, 100, 20, 200, 1, 4, 4, 1.0, 1.0, q_scale=2.0, seed=302)}[name]
    n_layers = 4
    seq_len, gamma = synth.draw_lengths(cfg)
    cu_q, _ = synth.prefix(gamma)
    n_q = int(cu_q[-1])
    kvs, qs, news = layer_inputs(cfg, n_layers, seq_len, n_q)
    bt = kvs[0].block_table                                   # same lengths, same seedless layout: one table
    for kv in kvs:
        assert kv.block_table.shape == bt.shape
    d_k = [dev_bf16(kv.k_pool) for kv in kvs]
    d_v = [dev_bf16(kv.v_pool) for kv in kvs]
    pools = [sv.spec_kv_pool_register(k, v) for k, v in zip(d_k, d_v)]
    d_q = [dev_bf16(q) for q in qs]
    d_o = [torch.zeros_like(q) for q in d_q]
    d_lse = [torch.zeros(q.shape[:2], dtype=torch.float32, device=DEV) for q in d_q]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    max_len = int(seq_len.max())
    ws = workspace(sv.spec_verify_attn_workspace_bytes(cfg.batch, cfg.gamma_max, cfg.hq, cfg.hkv, cfg.head_dim, max_len))
    launches = sv.sv_launch_count()
    sv.spec_verify_attn_layers(d_q, d_o, pools, dev(bt), dev(seq_len), dev(gamma), dev(cu_q), cfg.gamma_max, max_len,
                               ws, k_new=[dev_bf16(a) for a, _ in news] if append else None,
                               v_new=[dev_bf16(b) for _, b in news] if append else None, lses=d_lse,
                               device_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    if append:                                                # one append launch for all layers
        per_layer = (sv.sv_launch_count() - launches - 1) / n_layers
        assert per_layer in (1.0, 2.0)
    rows = used_rows(gamma, cu_q)
    scale = float(np.float32(cfg.head_dim ** -0.5))
    for l in range(n_layers):
        kp, vp = kvs[l].k_pool, kvs[l].v_pool
        if append:
            kp, vp = oracle.kv_append(news[l][0], news[l][1], kp, vp, kvs[l].strides, bt, seq_len, gamma, cu_q,
                                      cfg.page_size)
            np.testing.assert_array_equal(bits_of(d_k[l]), kp)     # whole pools, bit for bit
            np.testing.assert_array_equal(bits_of(d_v[l]), vp)
        o_ref, lse_ref = oracle.verify_attn(qs[l], kp, vp, kvs[l].strides, bt, seq_len, gamma, cu_q, cfg.hq, cfg.hkv,
                                            cfg.page_size, scale)
        o_gpu = synth.bf16_to_f32(bits_of(d_o[l])).astype(np.float64)
        assert np.abs(o_gpu[rows] - o_ref[rows]).max() <= ATTN_ATOL, l
        assert np.abs(np.expm1(d_lse[l].cpu().numpy().astype(np.float64)[rows] - lse_ref[rows])).max() <= 1e-5
    # the layers really differ: no two outputs alike
    assert not torch.equal(d_o[0], d_o[1])


def test_more_layers_than_one_append_launch_takes():
    cfg = synth.VerifyConfig("many", 2, 2, 1, 128, 100, 30, 60, 1, 2, 2, 1.0, 1.0, seed=303)
    n_layers = 27                                             # beyond the per-launch limit of the append
    seq_len, gamma = synth.draw_lengths(cfg)
    cu_q, _ = synth.prefix(gamma)
    n_q = int(cu_q[-1])
    kvs, qs, news = layer_inputs(cfg, n_layers, seq_len, n_q)
    bt = kvs[0].block_table
    d_k = [dev_bf16(kv.k_pool) for kv in kvs]
    d_v = [dev_bf16(kv.v_pool) for kv in kvs]
    pools = [sv.spec_kv_pool_register(k, v) for k, v in zip(d_k, d_v)]
    d_q = [dev_bf16(q) for q in qs]
    d_o = [torch.zeros_like(q) for q in d_q]
    max_len = int(seq_len.max())
    ws = workspace(sv.spec_verify_attn_workspace_bytes(cfg.batch, cfg.gamma_max, cfg.hq, cfg.hkv, cfg.head_dim, max_len))
    sv.spec_verify_attn_layers(d_q, d_o, pools, dev(bt), dev(seq_len), dev(gamma), dev(cu_q), cfg.gamma_max, max_len,
                               ws, k_new=[dev_bf16(a) for a, _ in news], v_new=[dev_bf16(b) for _, b in news])
    torch.cuda.synchronize()
    for l in (0, 23, 24, 26):
        kp, vp = oracle.kv_append(news[l][0], news[l][1], kvs[l].k_pool, kvs[l].v_pool, kvs[l].strides, bt, seq_len,
                                  gamma, cu_q, cfg.page_size)
        np.testing.assert_array_equal(bits_of(d_k[l]), kp)
        o_ref, _ = oracle.verify_attn(qs[l], kp, vp, kvs[l].strides, bt, seq_len, gamma, cu_q, cfg.hq, cfg.hkv,
                                      cfg.page_size, float(np.float32(cfg.head_dim ** -0.5)))
        o_gpu = synth.bf16_to_f32(bits_of(d_o[l])).astype(np.float64)
        rows = used_rows(gamma, cu_q)
        assert np.abs(o_gpu[rows] - o_ref[rows]).max() <= ATTN_ATOL


def test_host_errors():
    cfg = synth.VerifyConfig("err", 2, 4, 1, 128, 100, 100, 300, 2, 2, 2, 1.0, 1.0, seed=304)
    seq_len, gamma = synth.draw_lengths(cfg)
    cu_q, _ = synth.prefix(gamma)
    kvs, qs, news = layer_inputs(cfg, 2, seq_len, int(cu_q[-1]))
    pools = [sv.spec_kv_pool_register(dev_bf16(kv.k_pool), dev_bf16(kv.v_pool)) for kv in kvs]
    d_q = [dev_bf16(q) for q in qs]
    d_o = [torch.zeros_like(q) for q in d_q]
    args = (dev(kvs[0].block_table), dev(seq_len), dev(gamma), dev(cu_q), cfg.gamma_max, int(seq_len.max()))
    with pytest.raises(sv.SpecVerifyError) as e:      # workspace too small
        sv.spec_verify_attn_layers(d_q, d_o, pools, *args, workspace(16))
    assert e.value.status == sv.SV_EWORKSPACE
    with pytest.raises(sv.SpecVerifyError) as e:      # keys without values
        p = sv.attn_layers_params(d_q, d_o, pools, *args, k_new=[d_q[0][:, :1].contiguous()] * 2,
                                  v_new=[d_q[0][:, :1].contiguous()] * 2)
        p.v_new = None
        sv._check("spec_verify_attn_layers", sv.load().spec_verify_attn_layers(p, workspace(1 << 20).data_ptr(),
                                                                                  1 << 20, None))
    assert e.value.status == sv.SV_EINVAL
