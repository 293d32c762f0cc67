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


# ------------------------------------------------------------------ backward pass
def _rand_qkv(B, H, n, d, seed):
    rng = np.random.default_rng(seed)
    return tuple(rng.normal(size=(B, H, n, d)) for _ in range(4))      # Q, K, V, dO


@pytest.mark.parametrize("n,stride", [(7, 3), (12, 4), (9, 16)])
def test_backward_matches_central_differences(n, stride):
    Q, K, V, dO = _rand_qkv(1, 2, n, 5, 100 + n)
    dQ, dK, dV = att.strided_attention_bwd(Q, K, V, dO, stride)

    def loss(q, k, v):
        return float((att.strided_attention(q, k, v, stride)[0] * dO).sum())
    h = 1e-6
    rng = np.random.default_rng(5)
    for name, X, dX in (("q", Q, dQ), ("k", K, dK), ("v", V, dV)):
        for _ in range(25):
            idx = tuple(rng.integers(0, s) for s in X.shape)
            Xp, Xm = X.copy(), X.copy()
            Xp[idx] += h
            Xm[idx] -= h
            args_p = [Q, K, V]; args_m = [Q, K, V]
            j = "qkv".index(name)
            args_p[j], args_m[j] = Xp, Xm
            num = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(num - dX[idx]) <= 1e-6 * max(1.0, abs(num)), (name, idx)


def test_backward_directional_identity():
    # first-order change of <dO, Out> along a random direction equals the inner products with the gradients
    Q, K, V, dO = _rand_qkv(2, 3, 20, 8, 7)
    dq, dk, dv, _ = _rand_qkv(2, 3, 20, 8, 8)
    dQ, dK, dV = att.strided_attention_bwd(Q, K, V, dO, 6)
    eps = 1e-6
    f = lambda t: float((att.strided_attention(Q + t * dq, K + t * dk, V + t * dv, 6)[0] * dO).sum())
    num = (f(eps) - f(-eps)) / (2 * eps)
    ana = float((dQ * dq).sum() + (dK * dk).sum() + (dV * dv).sum())
    assert abs(num - ana) <= 1e-6 * max(1.0, abs(ana))


def test_backward_position_by_position_loop():
    # the same derivative written without matrices: one query position at a time, explicit key sets
    Q, K, V, dO = _rand_qkv(1, 1, 11, 4, 3)
    stride = 4
    n, d = 11, 4
    dQ = np.zeros((n, d)); dK = np.zeros((n, d)); dV = np.zeros((n, d))
    for i in range(n):
        js = [j for j in range(i + 1) if i - j < stride or (i - j) % stride == 0]
        s = np.array([Q[0, 0, i] @ K[0, 0, j] for j in js]) / np.sqrt(d)
        p = np.exp(s - s.max()); p /= p.sum()
        dp = np.array([dO[0, 0, i] @ V[0, 0, j] for j in js])
        ds = p * (dp - (p * dp).sum())
        for a, j in enumerate(js):
            dV[j] += p[a] * dO[0, 0, i]
            dQ[i] += ds[a] * K[0, 0, j] / np.sqrt(d)
            dK[j] += ds[a] * Q[0, 0, i] / np.sqrt(d)
    g = att.strided_attention_bwd(Q, K, V, dO, stride)
    np.testing.assert_allclose(g[0][0, 0], dQ, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g[1][0, 0], dK, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g[2][0, 0], dV, rtol=1e-12, atol=1e-12)


def test_backward_invariants():
    Q, K, V, dO = _rand_qkv(1, 2, 16, 4, 11)
    dQ, dK, dV = att.strided_attention_bwd(Q, K, V, dO, 5)
    # every row of P sums to one: the gradients of all values add up to the sum of the upstream gradients
    np.testing.assert_allclose(dV.sum(axis=-2), dO.sum(axis=-2), rtol=1e-12, atol=1e-12)
    # the first position attends only to itself: its softmax is constant, so its query gets no gradient
    np.testing.assert_allclose(dQ[..., 0, :], 0.0, atol=1e-15)
    # the last key is seen by the last query only
    np.testing.assert_allclose(dV[..., -1, :], dO[..., -1, :] * _p_last(Q, K, 5), rtol=1e-12)


def _p_last(Q, K, stride):
    n, d = Q.shape[-2], Q.shape[-1]
    i = n - 1
    js = [j for j in range(n) if i - j < stride or (i - j) % stride == 0]
    s = np.einsum("bhd,bhjd->bhj", Q[..., i, :], K[..., js, :]) / np.sqrt(d)
    p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    return p[..., -1:]          # weight of key n-1 in row n-1
