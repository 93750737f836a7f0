"""Pins for the oracle's attention: closed forms, special cases, a library softmax.

Each test is chosen so that a plausible slip in the oracle (wrong causal
offset, wrong head mapping, transposed strides, missing scale, page/slot mixed
up) fails at least one of them.
"""
import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

import oracle
from paper_2504_00030_b200 import synth


def _pool(rng, n_pages, hkv, ps, D):
    k = synth.bf16_bits(rng.standard_normal((n_pages, hkv, ps, D)).astype(np.float32))
    v = synth.bf16_bits(rng.standard_normal((n_pages, hkv, ps, D)).astype(np.float32))
    st = np.array([hkv * ps * D, ps * D, D, 1], np.int64)
    return k, v, st


def _library_attention(q, k_pool, v_pool, block_table, seq_len, gamma, cu_q, hq, hkv, ps, scale):
    """Independent restatement with numpy gathers + scipy's softmax + matmul."""
    qf = synth.bf16_to_f32(q).astype(np.float64)
    kf = synth.bf16_to_f32(k_pool).astype(np.float64)
    vf = synth.bf16_to_f32(v_pool).astype(np.float64)
    G = hq // hkv
    o = np.zeros(qf.shape)
    lse = np.zeros(qf.shape[:2])
    for b in range(len(seq_len)):
        L, R = int(seq_len[b]), int(gamma[b]) + 1
        n_pg = (L + ps - 1) // ps
        for h in range(hq):
            g = h // G
            K = kf[block_table[b, :n_pg], g].reshape(-1, kf.shape[-1])[:L]
            Vv = vf[block_table[b, :n_pg], g].reshape(-1, vf.shape[-1])[:L]
            for i in range(R):
                n = L - R + i + 1
                s = (K[:n] @ qf[cu_q[b] + i, h]) * scale
                o[cu_q[b] + i, h] = scipy_softmax(s) @ Vv[:n]
                lse[cu_q[b] + i, h] = np.log(np.sum(np.exp(s - s.max()))) + s.max()
    return o, lse


def test_single_key_returns_value_exactly():
    # L = R = 1: the only visible key is the row itself, softmax weight is 1, o = v_0.
    rng = np.random.default_rng(1)
    k, v, st = _pool(rng, 3, 2, 16, 64)
    q = synth.bf16_bits(rng.standard_normal((1, 4, 64)).astype(np.float32))
    bt = np.array([[2]], np.int32)
    o, lse = oracle.verify_attn(q, k, v, st, bt, [1], [0], [0, 1], 4, 2, 16, 0.125)
    for h in range(4):
        np.testing.assert_array_equal(o[0, h], synth.bf16_to_f32(v[2, h // 2, 0]).astype(np.float64))


def test_block_equal_to_context_is_causal_prefix():
    # L = R: row i sees exactly keys 0..i.  Row 0 must equal v_0; every row must
    # equal the single-row routine on the truncated sequence.
    rng = np.random.default_rng(2)
    k, v, st = _pool(rng, 2, 1, 16, 64)
    R = 9
    q = synth.bf16_bits(rng.standard_normal((R, 1, 64)).astype(np.float32))
    bt = np.array([[1, 0]], np.int32)
    o, lse = oracle.verify_attn(q, k, v, st, bt, [R], [R - 1], [0, R], 1, 1, 16, 0.125)
    np.testing.assert_array_equal(o[0, 0], synth.bf16_to_f32(v[1, 0, 0]).astype(np.float64))
    for i in range(R):
        oi, li = oracle.attn_row(q[i, 0], k, v, st, bt[0], 16, 0, i + 1, 0.125)
        np.testing.assert_array_equal(o[i, 0], oi)
        assert lse[i, 0] == li


def test_equal_keys_give_mean_of_values():
    rng = np.random.default_rng(3)
    k, v, st = _pool(rng, 4, 1, 16, 64)
    k[:] = k[0, 0, 0]           # every key identical -> uniform weights
    L, R = 50, 3
    q = synth.bf16_bits(rng.standard_normal((R, 1, 64)).astype(np.float32))
    bt = np.array([[3, 1, 0, 2]], np.int32)
    o, lse = oracle.verify_attn(q, k, v, st, bt, [L], [R - 1], [0, R], 1, 1, 16, 0.125)
    vf = synth.bf16_to_f32(v).astype(np.float64)
    vs = vf[bt[0], 0].reshape(-1, 64)
    for i in range(R):
        n = L - R + i + 1
        np.testing.assert_allclose(o[i, 0], vs[:n].mean(0), rtol=0, atol=1e-13)


def test_two_key_closed_form():
    # q = e_0, k_0 = 0, k_1 = e_0, scale = ln 3  ->  weights (1/4, 3/4), lse = ln 4.
    D = 64
    k = np.zeros((1, 1, 16, D), np.uint16)
    v = np.zeros((1, 1, 16, D), np.uint16)
    one = synth.bf16_bits(np.array([1.0], np.float32))[0]
    k[0, 0, 1, 0] = one
    v[0, 0, 0] = synth.bf16_bits(np.full(D, 2.0, np.float32))
    v[0, 0, 1] = synth.bf16_bits(np.full(D, -6.0, np.float32))
    q = np.zeros((1, 1, D), np.uint16)
    q[0, 0, 0] = one
    st = np.array([16 * D, 16 * D, D, 1], np.int64)
    o, lse = oracle.verify_attn(q, k, v, st, np.array([[0]], np.int32), [2], [0], [0, 1], 1, 1, 16,
                                np.log(3.0))
    np.testing.assert_allclose(o[0, 0], np.full(D, 0.25 * 2.0 + 0.75 * -6.0), rtol=1e-15)
    assert abs(lse[0, 0] - np.log(4.0)) < 1e-15


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2), (6, 1)])
def test_matches_library_softmax_ragged(hq, hkv):
    rng = np.random.default_rng(10 + hq)
    ps, D = 16, 32
    seq_len = np.array([1, 15, 16, 17, 40, 33], np.int32)
    gamma = np.array([0, 3, 15, 2, 5, 1], np.int32)
    cu_q, _ = synth.prefix(gamma)
    n_pages = int(((seq_len + ps - 1) // ps).sum())
    k, v, st = _pool(rng, n_pages + 2, hkv, ps, D)
    perm = rng.permutation(n_pages + 2).astype(np.int32)
    bt = np.full((len(seq_len), 3), -1, np.int32)
    at = 0
    for b, L in enumerate(seq_len):
        n = (L + ps - 1) // ps
        bt[b, :n] = perm[at:at + n]
        at += n
    q = synth.bf16_bits((3 * rng.standard_normal((cu_q[-1], hq, D))).astype(np.float32))
    scale = 1 / np.sqrt(D)
    o, lse = oracle.verify_attn(q, k, v, st, bt, seq_len, gamma, cu_q, hq, hkv, ps, scale)
    o2, lse2 = _library_attention(q, k, v, bt, seq_len, gamma, cu_q, hq, hkv, ps, scale)
    np.testing.assert_allclose(o, o2, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse2, rtol=0, atol=1e-12)


def test_page_permutation_is_bit_identical():
    rng = np.random.default_rng(5)
    ps, D, hkv = 16, 64, 2
    k, v, st = _pool(rng, 6, hkv, ps, D)
    bt = np.array([[0, 1, 2, 3]], np.int32)
    q = synth.bf16_bits(rng.standard_normal((4, 4, D)).astype(np.float32))
    args = ([60], [3], [0, 4], 4, hkv, ps, 0.125)
    o1, l1 = oracle.verify_attn(q, k, v, st, bt, *args)
    perm = np.array([4, 2, 5, 0, 1, 3])
    k2, v2 = np.empty_like(k), np.empty_like(v)
    k2[perm], v2[perm] = k, v            # physical page p moves to perm[p]
    o2, l2 = oracle.verify_attn(q, k2, v2, st, perm[bt].astype(np.int32), *args)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(l1, l2)


def test_gqa_equals_mha_with_replicated_heads():
    rng = np.random.default_rng(6)
    ps, D, hq, hkv = 16, 64, 8, 2
    k, v, st = _pool(rng, 3, hkv, ps, D)
    bt = np.array([[2, 0, 1]], np.int32)
    q = synth.bf16_bits(rng.standard_normal((3, hq, D)).astype(np.float32))
    o1, _ = oracle.verify_attn(q, k, v, st, bt, [44], [2], [0, 3], hq, hkv, ps, 0.125)
    krep, vrep = np.repeat(k, hq // hkv, axis=1), np.repeat(v, hq // hkv, axis=1)
    st2 = np.array([hq * ps * D, ps * D, D, 1], np.int64)
    o2, _ = oracle.verify_attn(q, krep, vrep, st2, bt, [44], [2], [0, 3], hq, hq, ps, 0.125)
    np.testing.assert_array_equal(o1, o2)


def test_strided_pool_layout():
    # [page, slot, head, dim] storage described only through the strides
    rng = np.random.default_rng(7)
    ps, D, hkv = 16, 64, 2
    k, v, st = _pool(rng, 3, hkv, ps, D)
    bt = np.array([[1, 2, 0]], np.int32)
    q = synth.bf16_bits(rng.standard_normal((2, 2, D)).astype(np.float32))
    o1, _ = oracle.verify_attn(q, k, v, st, bt, [40], [1], [0, 2], 2, hkv, ps, 0.125)
    kt = np.ascontiguousarray(k.transpose(0, 2, 1, 3))
    vt = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    st2 = np.array([ps * hkv * D, D, hkv * D, 1], np.int64)
    o2, _ = oracle.verify_attn(q, kt, vt, st2, bt, [40], [1], [0, 2], 2, hkv, ps, 0.125)
    np.testing.assert_array_equal(o1, o2)
