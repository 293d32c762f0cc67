"""Forward and input gradient on the 2:4 structured-sparse tensor-core path vs the CPU checker (needs a GPU).

The path splits W.M into the first two entries of every group of four contraction indices and a spill list; both
parts together are exact, so the results must meet the same tolerance as every other path for ANY mask.
"""
import numpy as np
import pytest

import mst_inputs
import oracle

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import TOL, dev, host, make_layer, rel_err, to_dev


def _conforming_mask(O, I, seed):
    """at most two entries in every aligned group of four input features (no spills in the forward product)"""
    rng = np.random.default_rng(seed)
    m = np.zeros((O, I), dtype=np.uint8)
    for g in range(0, I, 4):
        w = min(4, I - g)
        k = rng.integers(0, 3, size=O)
        order = np.argsort(rng.random((O, w)), axis=1)
        for o in range(O):
            m[o, g + order[o, : min(k[o], w)]] = 1
    return m


def _run(p, L, ldx=None, ldy=None):
    T, O, I = p.tokens, p.out_features, p.in_features
    X, dY = to_dev(p, "X", ldx), to_dev(p, "dY", ldy)
    ldx, ldy = ldx or I, ldy or O
    Y = torch.full((T, ldy), float("nan"), dtype=torch.bfloat16, device=dev())
    dX = torch.full((T, ldx), float("nan"), dtype=torch.bfloat16, device=dev())
    mst.mst_spmm_fwd(L.handle, X, ldx, T, Y, ldy)
    mst.mst_spmm_bwd_x(L.handle, dY, ldy, T, dX, ldx)
    torch.cuda.synchronize()
    return host(Y)[:, :O], host(dX)[:, :I]


@pytest.mark.parametrize("O,I,T,density,kind,pad", [
    (256, 128, 240, 0.3, "conforming", 0),   # one tile, no spills in the forward product
    (256, 128, 240, 0.1, "uniform", 0),
    (160, 200, 300, 0.2, "uniform", 0),      # ragged rows, contraction tail, token tail
    (130, 264, 513, 0.1, "uniform", 0),
    (128, 256, 256, 0.25, "uniform", 8),     # padded leading dimensions
    (520, 328, 900, 0.1, "uniform", 0),      # three row tiles, four token tiles
    (768, 768, 512, 0.06, "zipf", 0),        # saturated rows: groups with four entries, long spill lists
    (1024, 768, 1024, 0.25, "uniform", 0),   # the largest density the path accepts
    (64, 96, 17, 0.05, "uniform", 0),        # fewer tokens than one epilogue chunk
    (200, 96, 64, 0.0, "uniform", 0)])       # empty mask
def test_sparse_tc_products_match_oracle(O, I, T, density, kind, pad):
    if kind == "zipf":
        p = mst_inputs.zipf_layer("t", 3, O, I, T, "bf16", density, 2000 + O + I + T)
    else:
        p = mst_inputs.uniform_layer("t", 3, O, I, T, "bf16", density, 2000 + O + I + T)
        if kind == "conforming":
            p.mask[:] = _conforming_mask(O, I, 7)
    L = make_layer(p)
    L.set_path(mst.MST_PATH_SPARSE_TC)
    Wm = np.where(p.mask == 1, p.W, np.float32(0))
    Yr, dXr = oracle.fwd(p.X, Wm, p.mask), oracle.bwd_x(p.dY, Wm, p.mask)
    Y, dX = _run(p, L, I + pad if pad else None, O + pad if pad else None)
    assert rel_err(Y, Yr) <= TOL["bf16"]
    assert rel_err(dX, dXr) <= TOL["bf16"]
    # second call on the same structure (spill positions reused, values compressed again): identical bits
    Y2, dX2 = _run(p, L, I + pad if pad else None, O + pad if pad else None)
    np.testing.assert_array_equal(Y.view(np.uint32), Y2.view(np.uint32))
    np.testing.assert_array_equal(dX.view(np.uint32), dX2.view(np.uint32))
    assert mst.mst_device_error_flags() == 0
    L.close()


def test_sparse_tc_follows_value_changes_and_topology_updates():
    O, I, T = 384, 512, 500
    p = mst_inputs.uniform_layer("t", 1, O, I, T, "bf16", 0.12, 77)
    L = make_layer(p)
    L.set_path(mst.MST_PATH_SPARSE_TC)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    Y, dX = _run(p, L)
    assert rel_err(Y, oracle.fwd(p.X, W, M)) <= TOL["bf16"]
    # an optimizer step in place: every stored value doubled (exact in bf16)
    ptr, nnz = mst.mst_values(L.handle)
    assert nnz == p.nnz
    rp, ci, v = oracle.to_csr(W, M)
    v2 = (2.0 * v).astype(np.float32)
    bits = torch.from_numpy(mst_inputs.f32_to_bf16_bits(v2).view(np.int16)).to(dev())
    from cuda.bindings import runtime as cudart
    torch.cuda.synchronize()
    (err,) = cudart.cudaMemcpy(ptr, bits.data_ptr(), 2 * nnz, cudart.cudaMemcpyKind.cudaMemcpyDeviceToDevice)
    assert int(err) == 0
    W2 = (2.0 * W).astype(np.float32)
    Y, dX = _run(p, L)
    assert rel_err(Y, oracle.fwd(p.X, W2, M)) <= TOL["bf16"]
    assert rel_err(dX, oracle.bwd_x(p.dY, W2, M)) <= TOL["bf16"]
    # two topology updates: the spill positions are rebuilt for the new mask, grown weights are zero
    G = oracle.dense_grad(p.dY, p.X).astype(np.float32)
    Gd = torch.from_numpy(G).to(dev())
    for step in range(2):
        st = mst.mst_topology_update(L.handle, 0.3, -1, 0.25, 5, step, False, Gd)
        W2, M, *_ = oracle.mg_update(W2, M, G, st.n_prune, st.n_grad, st.n_rand, 5, step, p.layer_id)
        Y, dX = _run(p, L)
        assert rel_err(Y, oracle.fwd(p.X, W2, M)) <= TOL["bf16"]
        assert rel_err(dX, oracle.bwd_x(p.dY, W2, M)) <= TOL["bf16"]
    assert mst.mst_device_error_flags() == 0
    L.close()


def test_sparse_tc_request_on_a_dense_layer_falls_back():
    # more than a quarter of the entries active: the spill list could outgrow its buffer, the dense tiles are used
    p = mst_inputs.uniform_layer("t", 2, 192, 160, 300, "bf16", 0.6, 11)
    L = make_layer(p)
    L.set_path(mst.MST_PATH_SPARSE_TC)
    Wm = np.where(p.mask == 1, p.W, np.float32(0))
    Y, dX = _run(p, L)
    assert rel_err(Y, oracle.fwd(p.X, Wm, p.mask)) <= TOL["bf16"]
    assert rel_err(dX, oracle.bwd_x(p.dY, Wm, p.mask)) <= TOL["bf16"]
    L.close()
