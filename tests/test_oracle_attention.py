"""Pins for oracle/attention.py (O2): closed forms and the prefix-reuse == recompute identity."""
import math

import numpy as np

from oracle.attention import attend_batch, attend_request, attend_rows
from paper_2505_03756_b200 import synth


def _rand(seed, L, n, n_q=4, n_kv=2, d=8):
    rs = synth.Stream(seed, "att")
    return (rs.normal((n, n_q, d)).astype(np.float64), rs.normal((L, n_kv, d)).astype(np.float64),
            rs.normal((L, n_kv, d)).astype(np.float64))


def test_two_key_closed_form_and_causality():
    # d = 2, one head. keys k0 = (0,0), k1 = (1,0); q = (ln 3, 0): logits 0 and ln 3 -> weights 1/4, 3/4.
    q = np.array([[[math.log(3.0), 0.0]], [[math.log(3.0), 0.0]]])          # two new tokens
    k = np.array([[[0.0, 0.0]], [[1.0, 0.0]]])
    v = np.array([[[4.0, -8.0]], [[8.0, 0.0]]])
    o = attend_request(q, k, v, prefix_len=0, sm_scale=1.0)
    np.testing.assert_allclose(o[0, 0], [4.0, -8.0], atol=1e-15)             # token 0 sees only key 0
    np.testing.assert_allclose(o[1, 0], [0.25 * 4 + 0.75 * 8, 0.25 * -8.0], atol=1e-12)
    # with the first key cached (prefix_len = 1) the single new token sees both keys
    o = attend_request(q[:1], k, v, prefix_len=1, sm_scale=1.0)
    np.testing.assert_allclose(o[0, 0], [7.0, -2.0], atol=1e-12)
    # sm_scale multiplies the logits: scale 2 -> logit ln 9 -> weights 1/10, 9/10
    o = attend_request(q[:1], k, v, prefix_len=1, sm_scale=2.0)
    np.testing.assert_allclose(o[0, 0], [0.1 * 4 + 0.9 * 8, 0.1 * -8.0], atol=1e-12)


def test_prefix_reuse_equals_full_recompute():
    L, p = 37, 16
    q_all, k, v = _rand(7, L, L)
    full = attend_request(q_all, k, v, prefix_len=0, sm_scale=0.3)
    reuse = attend_request(q_all[p:], k, v, prefix_len=p, sm_scale=0.3)
    np.testing.assert_allclose(reuse, full[p:], rtol=1e-12, atol=1e-13)


def test_equal_values_and_equal_keys():
    q, k, v = _rand(8, 20, 5)
    v_same = np.broadcast_to(v[:1], v.shape).copy()
    o = attend_request(q, k, v_same, prefix_len=15, sm_scale=1.0)
    for h in range(4):
        np.testing.assert_allclose(o[:, h], np.broadcast_to(v[0, h // 2], (5, 8)), rtol=1e-12)
    k_same = np.broadcast_to(k[:1], k.shape).copy()
    o = attend_request(q, k_same, v, prefix_len=15, sm_scale=1.0)
    for j in range(5):
        for h in range(4):
            np.testing.assert_allclose(o[j, h], v[:15 + j + 1, h // 2].mean(axis=0), rtol=1e-12, atol=1e-13)


def test_single_key_and_weights_bounded():
    q, k, v = _rand(9, 1, 1)
    np.testing.assert_allclose(attend_request(q, k, v, 0, 1.0)[0, 3], v[0, 1], rtol=1e-15)
    q, k, v = _rand(10, 12, 4)
    o = attend_request(q, k, v, 8, 1.0)   # convex combination: inside the visible values' range
    for j in range(4):
        vis = v[:8 + j + 1, 0]
        assert np.all(o[j, 0] <= vis.max(axis=0) + 1e-12) and np.all(o[j, 0] >= vis.min(axis=0) - 1e-12)


def test_grouped_heads_equal_replicated_heads():
    q, k, v = _rand(11, 19, 6, n_q=6, n_kv=2)
    o_gqa = attend_request(q, k, v, 13, 0.5)
    o_mha = attend_request(q, np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1), 13, 0.5)
    np.testing.assert_allclose(o_gqa, o_mha, rtol=1e-13, atol=1e-14)


def test_softmax_shift_invariance_large_logits():
    # adding a constant vector to every key along q leaves the weights unchanged; no overflow at 1e4
    q, k, v = _rand(12, 9, 1, n_q=1, n_kv=1)
    o1 = attend_request(q, k, v, 8, 1.0)
    qn = q[0, 0] / np.dot(q[0, 0], q[0, 0])
    o2 = attend_request(q, k + 1e4 * qn, v, 8, 1.0)
    np.testing.assert_allclose(o1, o2, rtol=1e-6, atol=1e-8)


def test_rows_and_batch_forms_agree():
    q, k, v = _rand(13, 30, 10)
    full = attend_request(q, k, v, 20, 0.2)
    rows = attend_rows(q[[0, 9]], [20, 29], k, v, 0.2)
    np.testing.assert_allclose(rows, full[[0, 9]], rtol=1e-11, atol=1e-14)
    q2, k2, v2 = _rand(14, 5, 5)
    b = attend_batch(np.concatenate([q, q2]), [k, k2], [v, v2], [20, 0], [10, 5], 0.2)
    np.testing.assert_allclose(b[:10], full, rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(b[10:], attend_request(q2, k2, v2, 0, 0.2), rtol=1e-11, atol=1e-14)
    assert attend_batch(q[:0], [], [], [], [], 1.0).shape[0] == 0
    assert attend_request(q[:0], k, v, 30, 1.0).shape == (0, 4, 8)
