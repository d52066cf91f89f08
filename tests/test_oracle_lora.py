"""Pins for oracle/lora.py (O1): special cases, the dense closed form of Eq. 1, a hand-worked example."""
import numpy as np

from oracle.lora import lora_linear, lora_project
from paper_2505_03756_b200 import synth


def _case(seed=1, T=11, d_in=24, d_out=40, r=4, n_ad=3):
    rs = synth.Stream(seed, "t")
    x = synth.round_bf16(rs.normal((T, d_in)))
    yb = synth.round_bf16(rs.normal((T, d_out)))
    ad = {i: (synth.round_bf16(rs.normal((d_in, r), 0.5)), synth.round_bf16(rs.normal((r, d_out), 0.5)))
          for i in range(n_ad)}
    seg = np.array([0, 3, 4, 9, 11], dtype=np.int32)
    ids = np.array([2, 0, 1, 0], dtype=np.int32)
    return x, yb, ad, seg, ids


def test_hand_worked_integers():
    # one token x = [1, 2], A = [[1, 0], [0, 1]] (identity shrink), B = [[1, 2, 3], [4, 5, 6]], s = 2:
    # xA = [1, 2]; (xA)B = [1+8, 2+10, 3+12] = [9, 12, 15]; y = base + 2 * that.
    y = lora_project(np.array([[10., 20., 30.]]), np.array([[1., 2.]]), [0, 1], [7],
                     {7: (np.eye(2), np.array([[1., 2., 3.], [4., 5., 6.]]))}, 2.0)
    assert y.tolist() == [[28., 44., 60.]]
    # a non-symmetric shrink catches a transposed A: A = [[1, 2], [3, 4]], xA = [1+6, 2+8] = [7, 10]
    # (xA)B with B = [[1, 0], [0, 1]] = [7, 10]
    y = lora_project(np.zeros((1, 2)), np.array([[1., 2.]]), [0, 1], [0],
                     {0: (np.array([[1., 2.], [3., 4.]]), np.eye(2))}, 1.0)
    assert y.tolist() == [[7., 10.]]


def test_zero_branch_is_bit_exact_base():
    x, yb, ad, seg, ids = _case()
    zero = {i: (a, np.zeros_like(b)) for i, (a, b) in ad.items()}
    assert np.array_equal(lora_project(yb, x, seg, ids, zero, 2.0), yb.astype(np.float64))
    assert np.array_equal(lora_project(yb, x, seg, ids, ad, 0.0), yb.astype(np.float64))
    assert np.array_equal(lora_project(yb, x, seg, -np.ones_like(ids), ad, 2.0), yb.astype(np.float64))


def test_single_adapter_equals_dense_updated_weight():
    # Eq. 1: W' = W + s A B, y = x W'
    x, _, ad, _, _ = _case(seed=2)
    rs = synth.Stream(5, "w")
    W = rs.normal((x.shape[1], 40)).astype(np.float64)
    A, B = (m.astype(np.float64) for m in ad[1])
    s = 0.75
    dense = x.astype(np.float64) @ (W + s * (A @ B))
    got = lora_project(x.astype(np.float64) @ W, x, [0, x.shape[0]], [1], ad, s)
    np.testing.assert_allclose(got, dense, rtol=1e-12, atol=1e-12)


def test_per_segment_adapter_and_untouched_rows():
    x, yb, ad, seg, ids = _case(seed=3)
    ids = np.array([2, -1, 1, 0], dtype=np.int32)
    got = lora_project(yb, x, seg, ids, ad, 2.0)
    for s, lid in enumerate(ids):
        rows = slice(seg[s], seg[s + 1])
        if lid < 0:
            assert np.array_equal(got[rows], yb[rows].astype(np.float64))
        else:
            A, B = (m.astype(np.float64) for m in ad[int(lid)])
            # column-vector form of Eq. 2: (B^T A^T) x^T
            want = yb[rows] + 2.0 * (B.T @ (A.T @ x[rows].astype(np.float64).T)).T
            np.testing.assert_allclose(got[rows], want, rtol=1e-12, atol=1e-12)


def test_linear_in_scale_and_segment_permutation():
    x, yb, ad, seg, ids = _case(seed=4)
    z = np.zeros_like(yb)
    d1 = lora_project(z, x, seg, ids, ad, 1.0)
    d3 = lora_project(z, x, seg, ids, ad, 3.0)
    np.testing.assert_allclose(d3, 3.0 * d1, rtol=1e-12, atol=1e-14)
    # swap the first two segments (3 rows and 1 row): outputs move with their rows
    perm = np.concatenate([np.arange(3, 4), np.arange(0, 3), np.arange(4, 11)])
    seg2 = np.array([0, 1, 4, 9, 11], dtype=np.int32)
    ids2 = ids[[1, 0, 2, 3]]
    got = lora_project(yb[perm], x[perm], seg2, ids2, ad, 2.0)
    np.testing.assert_allclose(got, lora_project(yb, x, seg, ids, ad, 2.0)[perm], rtol=1e-13, atol=1e-13)


def test_empty_inputs():
    x, yb, ad, _, _ = _case()
    assert lora_project(yb[:0], x[:0], [0], [], ad, 2.0).shape == (0, yb.shape[1])
    got = lora_project(yb, x, [0, 0, 11], [1, 2], ad, 2.0)   # an empty segment in front
    np.testing.assert_allclose(got, lora_project(yb, x, [0, 11], [2], ad, 2.0))


def test_linear_with_base_weight_by_hand_and_against_the_updated_weight():
    # x = [1, 2], W = [[1, 2, 3], [4, 5, 6]] -> xW = [9, 12, 15]; A = [[1], [1]] -> xA = [3]; B = [[1, 0, -1]];
    # s = 2 -> y = [9 + 6, 12, 15 - 6]
    y = lora_linear(np.array([[1., 2.]]), np.array([[1., 2., 3.], [4., 5., 6.]]), [0, 1], [0],
                    {0: (np.array([[1.], [1.]]), np.array([[1., 0., -1.]]))}, 2.0)
    assert y.tolist() == [[15., 12., 9.]]
    # a segment without an adapter is the plain product
    y = lora_linear(np.array([[1., 2.]]), np.array([[1., 2., 3.], [4., 5., 6.]]), [0, 1], [-1], {}, 2.0)
    assert y.tolist() == [[9., 12., 15.]]
    # Eq. 1 per segment: rows of adapter i see W + s A_i B_i
    x, _, ad, seg, ids = _case(seed=6)
    W = synth.Stream(9, "w").normal((x.shape[1], 40)).astype(np.float64)
    got = lora_linear(x, W, seg, ids, ad, 0.5)
    for s_, lid in enumerate(ids):
        A, B = (m.astype(np.float64) for m in ad[int(lid)])
        rows = slice(seg[s_], seg[s_ + 1])
        np.testing.assert_allclose(got[rows], x[rows].astype(np.float64) @ (W + 0.5 * (A @ B)), rtol=1e-12, atol=1e-12)
