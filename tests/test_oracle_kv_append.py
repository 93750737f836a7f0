"""Pins of the oracle's cache append (the draft block's keys and values written behind the context
of a paged bf16 cache; KV caching, paper Section 5).  CPU only."""
import numpy as np
from scipy.special import softmax

import oracle
from paper_2504_00030_b200 import synth

SENTINEL = 0x40E0          # bf16 bits of 7.0: no N(0,1) draw rounds to it in these cases


def bits(rng, shape):
    return synth.bf16_bits(rng.standard_normal(shape).astype(np.float32))


def widen(b):
    return synth.bf16_to_f32(b).astype(np.float64)


def empty_pool(n_pages, hkv, D, slot_major=False):
    """A pool of sentinels and its strides, [page, head, slot, dim] or [page, slot, head, dim]."""
    if slot_major:
        pool = np.full((n_pages, 16, hkv, D), SENTINEL, np.uint16)
        strides = np.array([16 * hkv * D, D, hkv * D, 1], np.int64)
    else:
        pool = np.full((n_pages, hkv, 16, D), SENTINEL, np.uint16)
        strides = np.array([hkv * 16 * D, 16 * D, D, 1], np.int64)
    return pool, strides


def test_hand_worked_page_and_slot():
    # one sequence of 18 tokens whose last three are new: positions 15, 16, 17 -> the last slot of
    # its first page and the first two slots of its second page
    rng = np.random.default_rng(1)
    hkv, D = 2, 8
    kp, st = empty_pool(5, hkv, D)
    vp, _ = empty_pool(5, hkv, D)
    bt = np.array([[3, 1]], np.int32)
    kn, vn = bits(rng, (3, hkv, D)), bits(rng, (3, hkv, D))
    k2, v2 = oracle.kv_append(kn, vn, kp, vp, st, bt, [18], [2], [0, 3], 16)
    for g in range(hkv):
        np.testing.assert_array_equal(k2[3, g, 15], kn[0, g])
        np.testing.assert_array_equal(k2[1, g, 0], kn[1, g])
        np.testing.assert_array_equal(k2[1, g, 1], kn[2, g])
        np.testing.assert_array_equal(v2[3, g, 15], vn[0, g])
        np.testing.assert_array_equal(v2[1, g, 0], vn[1, g])
        np.testing.assert_array_equal(v2[1, g, 1], vn[2, g])
    # nothing else moved, and the arguments were not written
    assert (k2 != SENTINEL).sum() == 3 * hkv * D and (v2 != SENTINEL).sum() == 3 * hkv * D
    assert (kp == SENTINEL).all() and (vp == SENTINEL).all()


def dense_causal_attention(q, k, v, n_ctx, group):
    """Textbook attention of the last rows of a sequence: q [R, hq, D], k and v [L, hkv, D] float64;
    row i sees keys 0 .. n_ctx + i."""
    R, hq, D = q.shape
    o = np.zeros((R, hq, D))
    for i in range(R):
        for h in range(hq):
            g = h // group
            s = k[: n_ctx + i + 1, g] @ q[i, h] / np.sqrt(D)
            o[i, h] = softmax(s) @ v[: n_ctx + i + 1, g]
    return o


def test_attention_over_an_appended_cache_is_dense_attention():
    # context written as one block (the special case R = L), then a draft block appended behind it:
    # attention through the paged cache must equal textbook attention over the concatenation
    rng = np.random.default_rng(2)
    hq, hkv, D = 4, 2, 16
    L0 = np.array([37, 16, 5], np.int32)               # contexts: mid-page, exactly one page, short
    gam = np.array([4, 0, 11], np.int32)               # blocks that stay in a page, and that cross one
    B = len(L0)
    kp, st = empty_pool(12, hkv, D)
    vp, _ = empty_pool(12, hkv, D)
    bt = np.array([[7, 2, 9, 4], [0, 11, 5, -1], [6, 3, -1, -1]], np.int32)
    cu0 = np.concatenate([[0], np.cumsum(L0)]).astype(np.int32)
    k_ctx, v_ctx = bits(rng, (int(cu0[-1]), hkv, D)), bits(rng, (int(cu0[-1]), hkv, D))
    kp, vp = oracle.kv_append(k_ctx, v_ctx, kp, vp, st, bt, L0, L0 - 1, cu0, 16)
    cu_q = np.concatenate([[0], np.cumsum(gam + 1)]).astype(np.int32)
    k_new, v_new = bits(rng, (int(cu_q[-1]), hkv, D)), bits(rng, (int(cu_q[-1]), hkv, D))
    L = L0 + gam + 1
    kp, vp = oracle.kv_append(k_new, v_new, kp, vp, st, bt, L, gam, cu_q, 16)
    q = bits(rng, (int(cu_q[-1]), hq, D))
    o, _ = oracle.verify_attn(q, kp, vp, st, bt, L, gam, cu_q, hq, hkv, 16, D ** -0.5)
    for b in range(B):
        k = np.concatenate([widen(k_ctx[cu0[b]:cu0[b + 1]]), widen(k_new[cu_q[b]:cu_q[b + 1]])])
        v = np.concatenate([widen(v_ctx[cu0[b]:cu0[b + 1]]), widen(v_new[cu_q[b]:cu_q[b + 1]])])
        ref = dense_causal_attention(widen(q[cu_q[b]:cu_q[b + 1]]), k, v, int(L0[b]), hq // hkv)
        np.testing.assert_allclose(o[cu_q[b]:cu_q[b + 1]], ref, rtol=1e-12, atol=1e-14)
    # exactly the appended elements were written
    n_written = (int(cu0[-1]) + int(cu_q[-1])) * hkv * D
    assert (kp != SENTINEL).sum() == n_written and (vp != SENTINEL).sum() == n_written


def logical_view(pool, strides, bt_row, n_tokens, hkv, D):
    flat = pool.reshape(-1)
    out = np.zeros((n_tokens, hkv, D), np.uint16)
    for j in range(n_tokens):
        for g in range(hkv):
            at = int(bt_row[j // 16]) * strides[0] + g * strides[1] + (j % 16) * strides[2]
            out[j, g] = flat[at:at + D]
    return out


def test_layouts_and_page_permutations_hold_the_same_logical_cache():
    rng = np.random.default_rng(3)
    hkv, D = 3, 8
    gam = np.array([2, 6], np.int32)
    L = np.array([20, 39], np.int32)
    cu_q = np.array([0, 3, 10], np.int32)
    kn, vn = bits(rng, (10, hkv, D)), bits(rng, (10, hkv, D))
    bt = np.array([[1, 4, -1], [0, 5, 2]], np.int32)
    results = []
    for slot_major in (False, True):
        kp, st = empty_pool(6, hkv, D, slot_major)
        vp, _ = empty_pool(6, hkv, D, slot_major)
        k2, v2 = oracle.kv_append(kn, vn, kp, vp, st, bt, L, gam, cu_q, 16)
        results.append([(logical_view(k2, st, bt[b], L[b], hkv, D), logical_view(v2, st, bt[b], L[b], hkv, D))
                        for b in range(2)])
    perm = np.array([4, 2, 0, 5, 3, 1], np.int32)       # physical page p moves to perm[p]
    kp, st = empty_pool(6, hkv, D)
    vp, _ = empty_pool(6, hkv, D)
    bt2 = np.where(bt >= 0, perm[np.maximum(bt, 0)], -1).astype(np.int32)
    k3, v3 = oracle.kv_append(kn, vn, kp, vp, st, bt2, L, gam, cu_q, 16)
    results.append([(logical_view(k3, st, bt2[b], L[b], hkv, D), logical_view(v3, st, bt2[b], L[b], hkv, D))
                    for b in range(2)])
    for b in range(2):
        for other in results[1:]:
            np.testing.assert_array_equal(results[0][b][0], other[b][0])
            np.testing.assert_array_equal(results[0][b][1], other[b][1])
        # and the logical cache ends with the new rows, K and V not swapped
        R = gam[b] + 1
        np.testing.assert_array_equal(results[0][b][0][L[b] - R:], kn[cu_q[b]:cu_q[b] + R])
        np.testing.assert_array_equal(results[0][b][1][L[b] - R:], vn[cu_q[b]:cu_q[b] + R])
        assert (results[0][b][0][:L[b] - R] == SENTINEL).all()


def test_padded_row_slabs_write_only_the_rows_in_use():
    # every sequence owns gamma_max + 1 rows of the new-row arrays; rows beyond gamma[b] are not appended
    rng = np.random.default_rng(4)
    hkv, D, gmax = 2, 8, 5
    gam = np.array([1, 5, 0], np.int32)
    L = np.array([9, 30, 1], np.int32)
    cu_q, _ = synth.padded_offsets(3, gmax)
    kn, vn = bits(rng, (int(cu_q[-1]), hkv, D)), bits(rng, (int(cu_q[-1]), hkv, D))
    bt = np.array([[2, -1], [0, 3], [1, -1]], np.int32)
    kp, st = empty_pool(4, hkv, D)
    vp, _ = empty_pool(4, hkv, D)
    k2, _ = oracle.kv_append(kn, vn, kp, vp, st, bt, L, gam, cu_q, 16)
    assert (k2 != SENTINEL).sum() == int((gam + 1).sum()) * hkv * D
    np.testing.assert_array_equal(k2[1, :, 0], kn[cu_q[2]])          # the third sequence is its one new token
    np.testing.assert_array_equal(k2[2, :, 8], kn[cu_q[0] + 1])      # position 8 of the first sequence
