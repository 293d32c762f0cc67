"""Pins for the oracle's three products and the dense gradient (CPU only).

Each check ties the C++ triple loops to something that is not the oracle
itself: numpy's dense matmul on the materialised W*M, the all-ones special
case, the adjoint identity of the three products, and hand-computed values.
"""
import os

import numpy as np
import pytest

import oracle
from oracle import flop_model


def _rand_case(rng, T, O, I, density):
    X = rng.standard_normal((T, I))
    W = rng.standard_normal((O, I))
    dY = rng.standard_normal((T, O))
    M = (rng.random((O, I)) < density).astype(np.uint8)
    return X, W, dY, M


@pytest.mark.parametrize("T,O,I,density", [(5, 7, 9, 0.3), (3, 4, 6, 0.0), (4, 5, 3, 1.0), (17, 33, 65, 0.1),
                                           (1, 1, 1, 1.0), (6, 8, 8, 0.5)])
def test_products_equal_dense_matmul_on_masked_weights(T, O, I, density):
    rng = np.random.default_rng(100 + T * O * I)
    X, W, dY, M = _rand_case(rng, T, O, I, density)
    if 0.0 < density < 1.0 and O > 2 and I > 2:
        M[1, :] = 0          # an empty row
        M[:, 2] = 0          # an empty column
    Wm = W * M
    np.testing.assert_allclose(oracle.fwd(X, W, M), X @ Wm.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(oracle.bwd_x(dY, W, M), dY @ Wm, rtol=1e-12, atol=1e-12)
    G = dY.T @ X
    dW = oracle.dw(dY, X, M)
    np.testing.assert_allclose(dW, G * M, rtol=1e-12, atol=1e-12)
    assert np.all(dW[M == 0] == 0.0)                      # exactly zero, not merely small
    np.testing.assert_allclose(oracle.dense_grad(dY, X), G, rtol=1e-12, atol=1e-12)


def test_all_ones_mask_is_a_dense_gemm():
    rng = np.random.default_rng(7)
    X, W, dY, _ = _rand_case(rng, 9, 11, 13, 1.0)
    M = np.ones((11, 13), dtype=np.uint8)
    np.testing.assert_allclose(oracle.fwd(X, W, M), X @ W.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(oracle.bwd_x(dY, W, M), dY @ W, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(oracle.dw(dY, X, M), dY.T @ X, rtol=1e-12, atol=1e-12)


def test_hand_computed_example():
    # W = [[1,2,3],[4,5,6]], M keeps (0,0),(0,2),(1,1); X = [[1,10,100]]; dY = [[2,-1]]
    W = np.array([[1., 2., 3.], [4., 5., 6.]])
    M = np.array([[1, 0, 1], [0, 1, 0]], dtype=np.uint8)
    X = np.array([[1., 10., 100.]])
    dY = np.array([[2., -1.]])
    assert oracle.fwd(X, W, M).tolist() == [[301.0, 50.0]]            # 1*1+3*100 ; 5*10
    assert oracle.bwd_x(dY, W, M).tolist() == [[2.0, -5.0, 6.0]]      # 2*1 ; -1*5 ; 2*3
    assert oracle.dw(dY, X, M).tolist() == [[2.0, 0.0, 200.0], [0.0, -10.0, 0.0]]
    assert oracle.dense_grad(dY, X).tolist() == [[2.0, 20.0, 200.0], [-1.0, -10.0, -100.0]]


def test_adjoint_identity():
    # <Y, dY> = <X, dX> = <W.M, dW>: holds for any inputs; a transposed operand or wrong index breaks it.
    rng = np.random.default_rng(11)
    X, W, dY, M = _rand_case(rng, 12, 10, 14, 0.35)
    Y = oracle.fwd(X, W, M)
    dX = oracle.bwd_x(dY, W, M)
    dW = oracle.dw(dY, X, M)
    a, b, c = np.sum(Y * dY), np.sum(X * dX), np.sum(W * M * dW)
    assert abs(a - b) <= 1e-10 * abs(a) and abs(a - c) <= 1e-10 * abs(a)


def test_sampled_variants_match_full():
    rng = np.random.default_rng(13)
    X, W, dY, M = _rand_case(rng, 8, 6, 10, 0.4)
    Y, dX, G = oracle.fwd(X, W, M), oracle.bwd_x(dY, W, M), oracle.dense_grad(dY, X)
    t = np.array([0, 3, 7, 7]); o = np.array([5, 0, 2, 5]); i = np.array([9, 1, 0, 4])
    np.testing.assert_array_equal(oracle.fwd_at(X, W, M, t, o), Y[t, o])
    np.testing.assert_allclose(oracle.bwd_x_at(dY, W, M, t, i), dX[t, i], rtol=1e-13)
    np.testing.assert_array_equal(oracle.grad_at(dY, X, o, i), G[o, i])


def test_linearity_in_weights_and_mask_split():
    # Splitting the mask into two disjoint masks splits every product additively.
    rng = np.random.default_rng(17)
    X, W, dY, M = _rand_case(rng, 6, 9, 7, 0.6)
    sel = rng.random(M.shape) < 0.5
    Ma, Mb = (M * sel).astype(np.uint8), (M * ~sel).astype(np.uint8)
    np.testing.assert_allclose(oracle.fwd(X, W, Ma) + oracle.fwd(X, W, Mb), oracle.fwd(X, W, M), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(oracle.bwd_x(dY, W, Ma) + oracle.bwd_x(dY, W, Mb), oracle.bwd_x(dY, W, M), rtol=1e-12,
                               atol=1e-12)
    np.testing.assert_array_equal(oracle.dw(dY, X, Ma) + oracle.dw(dY, X, Mb), oracle.dw(dY, X, M))


# ------------------------------------------------------------ FLOP accounting
def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_flops.txt")
    out = {}
    with open(path) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def test_flop_model_reproduces_printed_totals():
    g = _golden()
    tiny = flop_model.training_flops(6, 384) / 1e9
    ss = flop_model.training_flops(12, 768, sparsity=0.8) / 1e9
    assert round(tiny, 1) == g["tiny_gflops"]
    assert round(ss, 1) == g["ss80_gflops"] == g["rigl80_gflops"]


def test_strided_attention_ratio_matches_printed_table():
    g = _golden()
    assert round(100 * flop_model.q_atten_strided(1024, 128), 2) == g["q_atten_strided_128_pct"]
    assert round(100 * flop_model.q_atten_strided(1024, 256), 2) == g["q_atten_strided_256_pct"]


def test_erdos_renyi_split_of_one_block():
    shapes = [(2304, 768), (768, 768), (3072, 768), (768, 3072)]
    d, eps = flop_model.erdos_renyi_densities(shapes, 0.04)
    total = sum(o * i for o, i in shapes)
    assert abs(sum(dl * o * i for dl, (o, i) in zip(d, shapes)) - 0.04 * total) < 1e-6
    assert abs(eps - 23.04) < 1e-9
    np.testing.assert_allclose(d, [0.04, 0.06, 0.0375, 0.0375], rtol=1e-12)
