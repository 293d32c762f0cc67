"""Pins for the oracle's strided sparse attention (CPU only)."""
import os

import numpy as np
import pytest

from oracle import attention as att


def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_flops.txt")
    out = {}
    with open(path) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def test_mask_population_matches_the_printed_ratios():
    # App. "FLOP calculation", table of sparse self-attention patterns: kept fraction of the n x n scores at n = 1024
    g = _golden()
    assert round(100.0 * att.strided_mask(1024, 256).sum() / 1024 ** 2, 2) == g["q_atten_strided_256_pct"]
    assert round(100.0 * att.strided_mask(1024, 128).sum() / 1024 ** 2, 2) == g["q_atten_strided_128_pct"]


def test_mask_shape_small():
    # stride 3: the three latest positions and every third one before them (the paper's figure uses l = 3)
    m = att.strided_mask(8, 3)
    assert m[7].tolist() == [False, True, False, False, True, True, True, True]
    assert m[2].tolist() == [True, True, True, False, False, False, False, False]
    assert not np.triu(m, 1).any() and m.diagonal().all()


def _causal_reference(Q, K, V):
    """Dense causal softmax attention written differently: explicit loops over positions, log-sum-exp form."""
    B, H, n, d = Q.shape
    out = np.zeros((B, H, n, d))
    for b in range(B):
        for h in range(H):
            for i in range(n):
                s = K[b, h, : i + 1] @ Q[b, h, i] / np.sqrt(d)
                lse = np.log(np.sum(np.exp(s - s.max()))) + s.max()
                out[b, h, i] = np.exp(s - lse) @ V[b, h, : i + 1]
    return out


def test_stride_at_least_n_is_causal_attention():
    rng = np.random.default_rng(3)
    Q, K, V = (rng.standard_normal((2, 3, 17, 8)) for _ in range(3))
    out, _ = att.strided_attention(Q, K, V, 17)
    np.testing.assert_allclose(out, _causal_reference(Q, K, V), rtol=1e-12, atol=1e-12)
    out2, _ = att.strided_attention(Q, K, V, 1000)
    np.testing.assert_allclose(out2, out, rtol=0, atol=0)


def test_constant_values_pass_through_and_first_row_copies_v0():
    rng = np.random.default_rng(4)
    Q, K = (rng.standard_normal((1, 2, 20, 4)) for _ in range(2))
    V = np.broadcast_to(np.array([1.0, -2.0, 0.5, 3.0]), (1, 2, 20, 4)).copy()
    out, _ = att.strided_attention(Q, K, V, 4)
    np.testing.assert_allclose(out, V, rtol=1e-13)
    V2 = rng.standard_normal((1, 2, 20, 4))
    out2, lse = att.strided_attention(Q, K, V2, 4)
    np.testing.assert_allclose(out2[:, :, 0], V2[:, :, 0], rtol=1e-13)        # position 0 attends to itself only
    np.testing.assert_allclose(lse[:, :, 0], np.einsum("bhd,bhd->bh", Q[:, :, 0], K[:, :, 0]) / 2.0, rtol=1e-13)


def test_hand_example_stride_2():
    # d = 1, all queries 0 -> uniform weights over S_i; stride 2, n = 5: S_4 = {4, 3} u {2, 0}
    Q = np.zeros((1, 1, 5, 1)); K = np.ones((1, 1, 5, 1))
    V = np.array([1.0, 10.0, 100.0, 1000.0, 10000.0]).reshape(1, 1, 5, 1)
    out, lse = att.strided_attention(Q, K, V, 2)
    np.testing.assert_allclose(out[0, 0, :, 0], [1.0, 5.5, 37.0, 370.0, 2775.25], rtol=1e-14)
    np.testing.assert_allclose(lse[0, 0], np.log([1, 2, 3, 3, 4]), rtol=1e-13)


@pytest.mark.parametrize("n,stride", [(9, 3), (16, 4), (13, 5), (6, 1)])
def test_matches_position_by_position_loop(n, stride):
    rng = np.random.default_rng(n * 31 + stride)
    Q, K, V = (rng.standard_normal((2, 2, n, 6)) for _ in range(3))
    out, _ = att.strided_attention(Q, K, V, stride)
    b, h, i = np.meshgrid(np.arange(2), np.arange(2), np.arange(n), indexing="ij")
    ref = att.strided_attention_at(Q, K, V, stride, b.ravel(), h.ravel(), i.ravel()).reshape(2, 2, n, 6)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-12)
    # a dropped key changes the result: attending without the strided part differs whenever it is non-empty
    if n > stride > 1:
        band = np.tril(np.ones((n, n), bool)) & ~np.tril(np.ones((n, n), bool), -stride)
        assert (att.strided_mask(n, stride) != band).any()
