"""CUDA library vs the CPU checker, element by element, on seeded inputs (needs a GPU)."""
import numpy as np
import pytest

import mst_inputs
import oracle

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import (TOL, dev, export_csc, export_csr, host, make_layer, mdtype, rel_err, tdtype, to_dev,
                          value_bits)


def _problem(O, I, T, dtype, density, seed, kind="uniform"):
    f = mst_inputs.uniform_layer if kind == "uniform" else mst_inputs.zipf_layer
    return f("t", seed % 7, O, I, T, dtype, density, seed)


# ----------------------------------------------------------------- structure
@pytest.mark.parametrize("O,I,dtype,density,kind", [
    (64, 64, "f32", 0.25, "uniform"), (130, 257, "bf16", 0.1, "uniform"), (33, 31, "f32", 0.5, "uniform"),
    (1, 1, "bf16", 1.0, "uniform"), (300, 200, "bf16", 0.0, "uniform"), (97, 160, "f32", 1.0, "uniform"),
    (768, 768, "bf16", 0.05, "zipf"), (5, 1000, "bf16", 0.3, "uniform"), (1000, 5, "f32", 0.3, "uniform")])
def test_pack_export_roundtrip(O, I, dtype, density, kind):
    p = _problem(O, I, 4, dtype, density, 100 + O + I, kind)
    L = make_layer(p)
    assert L.nnz == p.nnz
    L.validate()
    rp, ci, vb = export_csr(L, dtype)
    rp_r, ci_r, v_r = oracle.to_csr(p.W, p.mask)
    np.testing.assert_array_equal(rp, rp_r)
    np.testing.assert_array_equal(ci, ci_r)
    np.testing.assert_array_equal(vb, value_bits(v_r, dtype))
    # CSC view = CSR of the transpose; perm points back into CSR order
    cp, ri, pm = export_csc(L)
    cp_r, ri_r, _ = oracle.to_csr(p.W.T, p.mask.T)
    np.testing.assert_array_equal(cp, cp_r)
    np.testing.assert_array_equal(ri, ri_r)
    cols_of_csc = np.repeat(np.arange(I), np.diff(cp_r))
    np.testing.assert_array_equal(ci_r[pm], cols_of_csc)
    rows_of_csr = np.repeat(np.arange(O), np.diff(rp_r))
    np.testing.assert_array_equal(rows_of_csr[pm], ri_r)
    L.close()


def test_pack_capacity_and_padded_weights():
    p = _problem(40, 70, 4, "f32", 0.5, 9)
    L = mst.Layer(0, 40, 70, mst.MST_F32, p.nnz - 1)
    with pytest.raises(mst.MstError) as e:
        L.pack(to_dev(p, "W"), torch.from_numpy(p.mask).to(dev()))
    assert e.value.status == 4
    L.close()
    L = mst.Layer(0, 40, 70, mst.MST_F32, p.nnz)
    Wp = to_dev(p, "W", ld=96)
    L.pack(Wp, torch.from_numpy(p.mask).to(dev()), ldw=96)
    _, _, vb = export_csr(L, "f32")
    np.testing.assert_array_equal(vb, value_bits(oracle.to_csr(p.W, p.mask)[2], "f32"))
    L.close()


# ------------------------------------------------------------------ products
def _run_products(p, L, ldx=None, ldy=None):
    T, O, I = p.tokens, p.out_features, p.in_features
    X, dY = to_dev(p, "X", ldx), to_dev(p, "dY", ldy)
    ldx, ldy = ldx or I, ldy or O
    Y = torch.full((T, ldy), float("nan"), dtype=tdtype(p), device=dev())
    dX = torch.full((T, ldx), float("nan"), dtype=tdtype(p), device=dev())
    dW = torch.full((max(p.nnz, 1),), float("nan"), dtype=torch.float32, device=dev())
    G = torch.full((O, I), float("nan"), dtype=torch.float32, device=dev())
    mst.mst_spmm_fwd(L.handle, X, ldx, T, Y, ldy)
    mst.mst_spmm_bwd_x(L.handle, dY, ldy, T, dX, ldx)
    mst.mst_sddmm_dw(L.handle, dY, ldy, X, ldx, T, dW)
    mst.mst_dense_grad(dY, ldy, X, ldx, T, O, I, mdtype(p), G)
    torch.cuda.synchronize()
    return host(Y)[:, :O], host(dX)[:, :I], host(dW)[: p.nnz], host(G)


@pytest.mark.parametrize("O,I,T,dtype,density,kind,pad", [
    (160, 200, 300, "bf16", 0.2, "uniform", 0),      # several panels/chunks, ragged tails everywhere
    (160, 200, 300, "f32", 0.2, "uniform", 0),
    (130, 257, 513, "bf16", 0.1, "uniform", 0),      # odd sizes: scalar staging path
    (130, 257, 513, "f32", 0.1, "uniform", 0),
    (128, 256, 256, "bf16", 0.25, "uniform", 8),     # padded leading dimensions
    (64, 128, 1, "f32", 0.5, "uniform", 0),          # single token
    (200, 96, 700, "bf16", 1.0, "uniform", 0),       # all-ones mask
    (200, 96, 64, "bf16", 0.0, "uniform", 0),        # empty mask
    (768, 768, 512, "bf16", 0.06, "zipf", 0),        # skewed rows: some full, many empty
    (3, 5, 7, "f32", 0.6, "uniform", 0),
    (70, 1100, 260, "bf16", 0.15, "uniform", 0),
    (520, 328, 900, "bf16", 0.1, "uniform", 0),      # three N tiles / two K-tail blocks on the tensor-core path
    (1024, 768, 1024, "bf16", 0.05, "zipf", 0),
    (520, 328, 900, "bf16", 0.7, "uniform", 0),      # dense chunks of the sampled weight gradient: row-by-row stores
    (300, 1000, 2100, "bf16", 0.45, "uniform", 8),   # chunks on both sides of the row-by-row threshold
    (264, 520, 640, "bf16", 1.0, "uniform", 0)])     # all-ones mask over several tiles: the values are the dense image
def test_products_match_oracle(O, I, T, dtype, density, kind, pad):
    p = _problem(O, I, T, dtype, density, 1000 + O + I + T, kind)
    L = make_layer(p)
    tol = TOL[dtype]
    Wm = np.where(p.mask == 1, p.W, np.float32(0))
    Yr, dXr, Gr = oracle.fwd(p.X, Wm, p.mask), oracle.bwd_x(p.dY, Wm, p.mask), oracle.dense_grad(p.dY, p.X)
    rows, cols = np.nonzero(p.mask)
    # both kernel families: the sparse CUDA-core kernels and the dense-tile tensor-core kernels
    for path in (mst.MST_PATH_CUDA_CORE, mst.MST_PATH_TENSOR_CORE):
        L.set_path(path)
        Y, dX, dW, G = _run_products(p, L, I + pad if pad else None, O + pad if pad else None)
        assert rel_err(Y, Yr) <= tol, path
        assert rel_err(dX, dXr) <= tol, path
        assert rel_err(dW, Gr[rows, cols]) <= tol, path
        assert rel_err(G, Gr) <= tol, path
    assert mst.mst_device_error_flags() == 0
    L.close()


def test_results_are_run_to_run_identical():
    p = _problem(192, 320, 600, "bf16", 0.15, 77)
    L = make_layer(p)
    a = _run_products(p, L)
    b = _run_products(p, L)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x.view(np.uint32), y.view(np.uint32))
    L.close()


def test_step_host_matches_device_entry_points():
    p = _problem(160, 200, 300, "bf16", 0.2, 5)
    L = make_layer(p)
    Y, dX, dW, _ = _run_products(p, L)
    Xh = torch.from_numpy(p.X_bits.view(np.int16)).pin_memory()
    dYh = torch.from_numpy(p.dY_bits.view(np.int16)).pin_memory()
    Yh = torch.empty((300, 160), dtype=torch.int16).pin_memory()
    dXh = torch.empty((300, 200), dtype=torch.int16).pin_memory()
    dWh = torch.empty((p.nnz,), dtype=torch.float32).pin_memory()
    mst.mst_layer_step_host(L.handle, Xh, dYh, 300, Yh, dXh, dWh)
    np.testing.assert_array_equal(mst_inputs.bf16_bits_to_f32(Yh.numpy().view(np.uint16)), Y)
    np.testing.assert_array_equal(mst_inputs.bf16_bits_to_f32(dXh.numpy().view(np.uint16)), dX)
    np.testing.assert_array_equal(dWh.numpy(), dW)
    L.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("O,I,T,n_full", [(400, 1536, 300, 3), (1200, 2048, 520, 5), (97, 1024, 64, 1), (400, 768, 300, 3)])
def test_cuda_core_forward_splits_long_rows(O, I, T, n_full, dtype):
    # a few complete rows in an otherwise 3 % dense mask: the longest row is far above the mean, so the CUDA-core
    # forward hands the long rows (a thousand entries or more; the last case stays below that) to several warps; same
    # results as the checker, identical bits from run to run
    p = _problem(O, I, T, dtype, 0.03, 5200 + O, "uniform")
    rng = np.random.default_rng(O + T)
    full = rng.choice(O, size=n_full, replace=False)
    p.mask[full, :] = 1
    p.mask[full[0], ::3] = 0                       # one long row that is not complete
    L = make_layer(p)
    L.set_path(mst.MST_PATH_CUDA_CORE)
    Wm = np.where(p.mask == 1, p.W, np.float32(0))
    X = to_dev(p, "X")
    outs = []
    for rep in range(2):
        Y = torch.full((T, O), float("nan"), dtype=tdtype(p), device=dev())
        mst.mst_spmm_fwd(L.handle, X, I, T, Y, O)
        torch.cuda.synchronize()
        outs.append(host(Y))
    assert rel_err(outs[0], oracle.fwd(p.X, Wm, p.mask)) <= TOL[dtype]
    np.testing.assert_array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))
    assert mst.mst_device_error_flags() == 0
    L.close()


# ------------------------------------------------------------ topology update
def _update_both(L, p, W, M, G, zeta, target, R, seed, step, allow=False):
    """Run one update on the GPU and in the oracle from the same state; compare bit-exactly."""
    O, I = M.shape
    Gd = None if G is None else torch.from_numpy(G).to(dev())
    st = mst.mst_topology_update(L.handle, zeta, target, R, seed, step, allow, Gd)
    n_prune, n_grow, n_rand, n_grad = oracle.mg_counts(zeta, int(M.sum()), target, O * I, R)
    assert (st.n_prune, st.n_rand, st.n_grad) == (n_prune, n_rand, n_grad)
    Wn, Mn, *_ = oracle.mg_update(W, M, G, n_prune, n_grad, n_rand, seed, step, p.layer_id, allow)
    assert st.nnz_after == int(Mn.sum()) == L.nnz
    assert st.max_row_nnz == int(Mn.sum(1).max())
    rp, ci, vb = export_csr(L, p.dtype)
    rp_r, ci_r, v_r = oracle.to_csr(Wn, Mn)
    np.testing.assert_array_equal(rp, rp_r)
    np.testing.assert_array_equal(ci, ci_r)
    np.testing.assert_array_equal(vb, value_bits(v_r, p.dtype))
    L.validate()
    return Wn, Mn


def _set_update_variant(monkeypatch, variant):
    env = {"fused": {}, "phases": {"MST_UPDATE_FUSED": "0"}, "fused_sequential": {"MST_UPDATE_DUAL": "0"},
           "fused_bracket_miss": {"MST_UPDATE_RAND_SIGMAS": "0.001"}, "fused_no_bracket": {"MST_UPDATE_RAND_SIGMAS": "0"},
           "fused_no_key_cache": {"MST_UPDATE_NO_SMEM_KEYS": "1"}}[variant]
    for k in ("MST_UPDATE_FUSED", "MST_UPDATE_DUAL", "MST_UPDATE_RAND_SIGMAS", "MST_UPDATE_NO_SMEM_KEYS"):
        monkeypatch.delenv(k, raising=False)
    for k, v in env.items():
        monkeypatch.setenv(k, v)             # read by the library at every call


@pytest.mark.parametrize("variant", ["fused", "fused_no_key_cache", "fused_bracket_miss", "fused_sequential"])
def test_update_of_a_layer_beyond_the_register_key_cache(variant, monkeypatch):
    # 2.6 M entries: a block's slice no longer fits the key registers; keys live in shared memory or are recomputed
    _set_update_variant(monkeypatch, variant)
    O, I = 1024, 2560
    p = _problem(O, I, 4, "bf16", 0.05, 4100, "uniform")
    L = make_layer(p)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    rng = np.random.default_rng(9)
    for step in range(3):
        G = rng.standard_normal((O, I)).astype(np.float32)
        G.reshape(-1)[::7] = np.float32(0.125)
        W, M = _update_both(L, p, W, M, G, 0.3, -1, 0.25, 11, step)
    L.close()


@pytest.mark.parametrize("O,I,dtype,density,kind,zeta,R,allow", [
    (96, 160, "f32", 0.25, "uniform", 0.3, 0.25, False), (130, 257, "bf16", 0.1, "uniform", 0.3, 0.25, False),
    (256, 512, "bf16", 0.05, "zipf", 0.1, 0.25, False), (64, 96, "f32", 0.3, "uniform", 0.3, 0.0, False),
    (64, 96, "bf16", 0.3, "uniform", 0.3, 1.0, False), (96, 160, "bf16", 0.25, "uniform", 0.5, 0.25, True),
    (33, 31, "f32", 0.5, "uniform", 1.0, 0.5, False)])
@pytest.mark.parametrize("variant", ["fused", "phases", "fused_sequential", "fused_bracket_miss", "fused_no_bracket"])
def test_update_is_bit_exact_over_consecutive_steps(O, I, dtype, density, kind, zeta, R, allow, variant, monkeypatch):
    # every implementation of the update: the single cooperative kernel (prune and gradient selections side by side,
    # random growth by bracket), the kernel-per-phase sequence, the cooperative kernel with one selection after the
    # other, with a bracket so narrow that it usually misses (general radix select takes over), and without bracket
    _set_update_variant(monkeypatch, variant)
    p = _problem(O, I, 4, dtype, density, 300 + O + I, kind)
    L = make_layer(p)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    rng = np.random.default_rng(O * I)
    for step in range(4):     # grown weights are +0: from the second step on, ties at |w| = 0 decide the pruning
        G = rng.standard_normal((O, I)).astype(np.float32)
        G.reshape(-1)[::3] = np.float32(0.25)        # ties among gradient magnitudes
        G.reshape(-1)[1::5] = np.float32(-0.25)
        W, M = _update_both(L, p, W, M, G, zeta, -1, R, 42, step, allow)
    L.close()


def test_update_of_a_larger_layer_after_a_small_one_with_another_form():
    # the cooperative kernel's shared-memory limit is a property of the function, not of a launch: a small layer updated
    # with the key cache in shared memory must not leave a limit behind that a later, larger layer (updated with
    # regrowth of just-pruned links, hence one selection after the other and no key cache) exceeds
    small = _problem(33, 95, 4, "bf16", 0.3, 61)
    Ls = make_layer(small)
    Ws = np.where(small.mask == 1, small.W, np.float32(0)).astype(np.float32)
    _update_both(Ls, small, Ws, small.mask.copy(), np.ones((33, 95), np.float32), 0.3, -1, 0.25, 3, 0)
    big = _problem(794, 865, 4, "bf16", 0.0, 62)
    Lb = make_layer(big)
    rng = np.random.default_rng(4)
    G = rng.standard_normal((794, 865)).astype(np.float32)
    Wb = np.zeros((794, 865), np.float32)
    _update_both(Lb, big, Wb, big.mask.copy(), G, 0.3, 170320, 0.25, 3, 0, allow=True)     # growth from an empty mask
    Ls.close()
    Lb.close()


def test_update_changes_density_both_ways_and_reaches_dense_and_empty():
    O, I = 80, 96
    p = _problem(O, I, 4, "bf16", 0.3, 55)
    L = make_layer(p)        # capacity = O*I
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    rng = np.random.default_rng(1)
    for step, frac in enumerate([0.1, 0.04, 0.5, 1.0, 0.2, 0.0, 0.3]):
        G = rng.standard_normal((O, I)).astype(np.float32)
        W, M = _update_both(L, p, W, M, G, 0.3, int(round(frac * O * I)), 0.25, 7, step)
    L.close()


def test_fused_update_tie_rank_scans_do_not_share_partial_sums():
    """Two grid-wide scans with no barrier of their own between them (a tie-rank scan directly followed by the scan of
    the new mask) must not share their per-block partial sums.  Pure-prune updates of a bf16 layer (prune keys tie all
    the time) and R = 0 updates on a gradient with few distinct magnitudes, many iterations, bit-exact each time."""
    O, I = 768, 768          # enough mask words for a full-size cooperative grid
    p = _problem(O, I, 4, "bf16", 0.5, 901)
    L = make_layer(p)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    W = mst_inputs.bf16_bits_to_f32((mst_inputs.f32_to_bf16_bits(W) & np.uint16(0xFF80)))   # 1 mantissa bit: heavy ties
    Wd = torch.from_numpy(mst_inputs.f32_to_bf16_bits(W).view(np.int16)).to(dev()).view(torch.bfloat16)
    L.pack(Wd, torch.from_numpy(p.mask).to(dev()))
    M = p.mask.copy()
    nnz = int(M.sum())
    for step in range(12):   # warm-up style: prune only, the target shrinks every step
        nnz = int(nnz * 0.93)
        W, M = _update_both(L, p, W, M, None, 0.05, nnz, 0.0, 5, step)
    rng = np.random.default_rng(17)
    for step in range(12):   # R = 0 on a gradient with four distinct magnitudes
        G = rng.choice(np.array([0.5, -0.5, 0.25, -1.0], dtype=np.float32), size=(O, I))
        W, M = _update_both(L, p, W, M, G, 0.3, -1, 0.0, 5, 100 + step)
    L.close()


def test_rejected_update_leaves_the_layer_unchanged():
    p = _problem(64, 96, 4, "bf16", 0.25, 77)
    L = make_layer(p)
    rp0, ci0, vb0 = export_csr(L, p.dtype)
    G = torch.zeros(64, 96, device=dev())
    o, i = np.argwhere(p.mask == 0)[5]
    G[o, i] = float("inf")
    with pytest.raises(mst.MstError) as e:
        mst.mst_topology_update(L.handle, 0.3, -1, 0.25, 0, 0, False, G)
    assert e.value.status == 6
    assert L.nnz == p.nnz
    rp1, ci1, vb1 = export_csr(L, p.dtype)
    np.testing.assert_array_equal(rp0, rp1)
    np.testing.assert_array_equal(ci0, ci1)
    np.testing.assert_array_equal(vb0, vb1)
    L.validate()                                   # the flag was reported once and is clear again; CSC view rebuilt
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    _update_both(L, p, W, p.mask.copy(), np.ones((64, 96), np.float32), 0.3, -1, 0.25, 0, 1)   # a good update still works
    L.close()


def test_update_without_gradient_and_identity():
    p = _problem(64, 64, 4, "f32", 0.25, 66)
    L = make_layer(p)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    W, M = _update_both(L, p, W, M, None, 0.3, -1, 1.0, 3, 0)          # SET rule needs no gradient
    W2, M2 = _update_both(L, p, W, M, None, 0.0, -1, 0.25, 3, 1)       # zeta = 0: nothing changes
    np.testing.assert_array_equal(M2, M)
    L.close()


def test_error_statuses():
    p = _problem(32, 32, 4, "f32", 0.25, 8)
    # unpacked layer
    L = mst.Layer(0, 32, 32, mst.MST_F32)
    with pytest.raises(mst.MstError) as e:
        mst.mst_layer_nnz(L.handle)
    assert e.value.status == 9
    L.close()
    with pytest.raises(mst.MstError) as e:
        mst.mst_layer_create(0, 0, 32, mst.MST_F32, 10)
    assert e.value.status == 2
    with pytest.raises(mst.MstError) as e:
        mst.mst_layer_create(0, 32, 32, 5, 10)
    assert e.value.status == 3
    with pytest.raises(mst.MstError) as e:
        mst.mst_layer_create(0, 32, 32, mst.MST_F32, 32 * 32 + 1)
    assert e.value.status == 4
    L = make_layer(p, capacity=p.nnz + 10)
    X = to_dev(p, "X")
    Y = torch.empty(4, 32, device=dev())
    with pytest.raises(mst.MstError) as e:
        mst.mst_spmm_fwd(L.handle, X, 16, 4, Y, 32)          # leading dimension too small
    assert e.value.status == 2
    with pytest.raises(mst.MstError) as e:
        mst.mst_spmm_fwd(L.handle, None, 32, 4, Y, 32)
    assert e.value.status == 1
    G = torch.zeros(32, 32, device=dev())
    with pytest.raises(mst.MstError) as e:
        mst.mst_topology_update(L.handle, 0.3, p.nnz + 11, 0.25, 0, 0, False, G)     # beyond capacity
    assert e.value.status == 4
    with pytest.raises(mst.MstError) as e:
        mst.mst_topology_update(L.handle, 0.3, 32 * 32 + 1, 0.25, 0, 0, False, G)    # beyond the layer
    assert e.value.status == 5
    with pytest.raises(mst.MstError) as e:
        mst.mst_topology_update(L.handle, 1.5, -1, 0.25, 0, 0, False, G)
    assert e.value.status == 1
    with pytest.raises(mst.MstError) as e:
        mst.mst_topology_update(L.handle, 0.3, -1, 0.25, 0, 0, False, None)          # gradient growth without G
    assert e.value.status == 1
    G[3, 4] = float("nan")
    if p.mask[3, 4] == 0:
        with pytest.raises(mst.MstError) as e:
            mst.mst_topology_update(L.handle, 0.3, -1, 0.25, 0, 0, False, G)
        assert e.value.status == 6
    L.close()


# ------------------------------------------------------- tensor-core dense gradient
@pytest.mark.parametrize("O,I,T", [(300, 520, 1000), (512, 512, 4096), (128, 256, 64), (136, 264, 72), (1024, 768, 2048)])
def test_dense_grad_tensor_core_path(O, I, T):
    # bf16 with 16-byte-aligned rows takes the tcgen05 contraction: several tiles, ragged tails in M, N and K,
    # token-range splitting with the fixed-order reduction
    p = _problem(O, I, T, "bf16", 0.1, 4000 + O + I + T)
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    G = torch.full((O, I), float("nan"), dtype=torch.float32, device=dev())
    mst.mst_dense_grad(dY, O, X, I, T, O, I, mst.MST_BF16, G)
    G2 = torch.full((O, I), float("nan"), dtype=torch.float32, device=dev())
    mst.mst_dense_grad(dY, O, X, I, T, O, I, mst.MST_BF16, G2)
    assert mst.mst_device_error_flags() == 0
    Gr = oracle.dense_grad(p.dY, p.X)
    assert rel_err(host(G), Gr) <= 1e-5          # exact bf16 products, fp32 accumulation
    np.testing.assert_array_equal(host(G).view(np.uint32), host(G2).view(np.uint32))     # deterministic


@pytest.mark.parametrize("O,I,T,dtype", [(300, 520, 1000, "bf16"), (130, 257, 200, "f32"), (512, 512, 2048, "bf16")])
def test_dense_grad_dw_gives_both_gradients(O, I, T, dtype):
    p = _problem(O, I, T, dtype, 0.15, 6000 + O + I)
    L = make_layer(p)
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    G = torch.full((O, I), float("nan"), dtype=torch.float32, device=dev())
    dW = torch.full((p.nnz,), float("nan"), dtype=torch.float32, device=dev())
    L.dense_grad_dw(dY, X, T, G, dW)
    torch.cuda.synchronize()
    Gr = oracle.dense_grad(p.dY, p.X)
    rows, cols = np.nonzero(p.mask)
    assert rel_err(host(G), Gr) <= TOL[dtype]
    assert rel_err(host(dW), Gr[rows, cols]) <= TOL[dtype]
    np.testing.assert_array_equal(host(dW), host(G)[rows, cols])        # exactly the sampled entries of G
    L.close()


@pytest.mark.parametrize("dtype,fused", [("bf16", "1"), ("f32", "1"), ("bf16", "0")])
def test_mest_prune_criterion_is_bit_exact(dtype, fused, monkeypatch):
    # prune key |theta| + lambda |grad| (scheme table, MEST column), formed in fp32 on both sides
    monkeypatch.setenv("MST_UPDATE_FUSED", fused)
    O, I = 96, 160
    p = _problem(O, I, 4, dtype, 0.3, 7100)
    L = make_layer(p)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    rng = np.random.default_rng(3)
    for step in range(3):
        G = (rng.standard_normal((O, I)) * 0.05).astype(np.float32)
        st = mst.mst_topology_update(L.handle, 0.3, -1, 0.25, 5, step, False, torch.from_numpy(G).to(dev()),
                                     prune_grad_weight=0.5)
        c = oracle.mg_counts(0.3, int(M.sum()), -1, O * I, 0.25)
        W, M, *_ = oracle.mg_update(W, M, G, c[0], c[3], c[2], 5, step, p.layer_id, False, 0.5)
        rp, ci, vb = export_csr(L, dtype)
        rp_r, ci_r, v_r = oracle.to_csr(W, M)
        np.testing.assert_array_equal(rp, rp_r)
        np.testing.assert_array_equal(ci, ci_r)
        np.testing.assert_array_equal(vb, value_bits(v_r, dtype))
    L.close()


def test_async_host_step_overlaps_layers_and_matches():
    probs = [_problem(160, 200, 300, "bf16", 0.2, 8100), _problem(96, 256, 300, "bf16", 0.1, 8200)]
    layers, bufs, want = [], [], []
    for p in probs:
        L = make_layer(p)
        want.append(_run_products(p, L)[:3])
        T, O, I = p.tokens, p.out_features, p.in_features
        b = dict(X=torch.from_numpy(p.X_bits.view(np.int16)).pin_memory(), dY=torch.from_numpy(p.dY_bits.view(np.int16)).pin_memory(),
                 Y=torch.empty((T, O), dtype=torch.int16).pin_memory(), dX=torch.empty((T, I), dtype=torch.int16).pin_memory(),
                 dW=torch.empty((p.nnz,), dtype=torch.float32).pin_memory())
        layers.append(L); bufs.append(b)
    for rep in range(2):                       # the second round reuses the staging buffers of the first
        for p, L, b in zip(probs, layers, bufs):
            b["Y"].zero_(); b["dX"].zero_(); b["dW"].zero_()
            mst.mst_layer_step_host_async(L.handle, b["X"], b["dY"], p.tokens, b["Y"], b["dX"], b["dW"])
        for L in layers:
            mst.mst_layer_step_host_wait(L.handle)
        for (Y, dX, dW), b in zip(want, bufs):
            np.testing.assert_array_equal(mst_inputs.bf16_bits_to_f32(b["Y"].numpy().view(np.uint16)), Y)
            np.testing.assert_array_equal(mst_inputs.bf16_bits_to_f32(b["dX"].numpy().view(np.uint16)), dX)
            np.testing.assert_array_equal(b["dW"].numpy(), dW)
    for L in layers:
        L.close()


def test_async_host_steps_back_to_back_without_waiting():
    # three steps of one layer issued without a wait in between, each with its own inputs and result buffers: a
    # step's inputs arrive while the previous step's results leave, and no staging buffer is reused too early
    O, I, T = 512, 768, 2048          # large enough that the copies and the kernels really overlap
    steps = []
    L = None
    for k in range(3):
        p = _problem(O, I, T, "bf16", 0.2, 8300 + k)
        if L is None:
            p0, L = p, make_layer(p)
        q = mst_inputs.make_layer(p0.name, p0.layer_id, O, I, T, "bf16", p0.mask, 8300 + k)   # same weights' mask, new X / dY
        q.W, q.W_bits = p0.W, p0.W_bits
        want = _run_products(q, L)[:3]
        b = dict(X=torch.from_numpy(q.X_bits.view(np.int16)).pin_memory(), dY=torch.from_numpy(q.dY_bits.view(np.int16)).pin_memory(),
                 Y=torch.zeros((T, O), dtype=torch.int16).pin_memory(), dX=torch.zeros((T, I), dtype=torch.int16).pin_memory(),
                 dW=torch.zeros((p0.nnz,), dtype=torch.float32).pin_memory())
        steps.append((want, b))
    for _, b in steps:
        mst.mst_layer_step_host_async(L.handle, b["X"], b["dY"], T, b["Y"], b["dX"], b["dW"])
    mst.mst_layer_step_host_wait(L.handle)      # the latest step; the earlier ones precede it on the same streams
    torch.cuda.synchronize()
    for (Y, dX, dW), b in steps:
        np.testing.assert_array_equal(mst_inputs.bf16_bits_to_f32(b["Y"].numpy().view(np.uint16)), Y)
        np.testing.assert_array_equal(mst_inputs.bf16_bits_to_f32(b["dX"].numpy().view(np.uint16)), dX)
        np.testing.assert_array_equal(b["dW"].numpy(), dW)
    assert mst.mst_device_error_flags() == 0
    L.close()


@pytest.mark.parametrize("T", [0, 1, 127, 129])
def test_token_count_edges_on_the_tensor_path(T):
    O, I = 256, 192
    p = _problem(O, I, max(T, 1), "bf16", 0.2, 9000 + T)
    L = make_layer(p)
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    Y = torch.full((max(T, 1), O), 7.0, dtype=torch.bfloat16, device=dev())
    dX = torch.full((max(T, 1), I), 7.0, dtype=torch.bfloat16, device=dev())
    dW = torch.full((p.nnz,), 7.0, dtype=torch.float32, device=dev())
    G = torch.full((O, I), 7.0, dtype=torch.float32, device=dev())
    L.fwd(X, Y, T); L.bwd_x(dY, dX, T); L.sddmm(dY, X, T, dW); L.dense_grad(dY, X, T, G)
    torch.cuda.synchronize()
    if T == 0:                                  # nothing to contract: gradients are zero, activations untouched
        assert float(dW.abs().max()) == 0.0 and float(G.abs().max()) == 0.0
        assert float(Y.float().min()) == 7.0 and float(dX.float().min()) == 7.0
    else:
        Wm = np.where(p.mask == 1, p.W, np.float32(0))
        Xs, dYs = p.X[:T], p.dY[:T]
        assert rel_err(host(Y)[:T], oracle.fwd(Xs, Wm, p.mask)) <= TOL["bf16"]
        assert rel_err(host(dX)[:T], oracle.bwd_x(dYs, Wm, p.mask)) <= TOL["bf16"]
        Gr = oracle.dense_grad(dYs, Xs)
        rows, cols = np.nonzero(p.mask)
        assert rel_err(host(dW), Gr[rows, cols]) <= TOL["bf16"]
        assert rel_err(host(G), Gr) <= TOL["bf16"]
    assert mst.mst_device_error_flags() == 0
    L.close()


@pytest.mark.parametrize("O,I,T", [(520, 328, 900), (136, 264, 72), (768, 3072, 1000), (100, 64, 33)])
def test_staged_and_direct_stores_agree(O, I, T, monkeypatch):
    # the contraction's rows leave either through shared memory and TMA stores (default) or by per-thread stores;
    # both must write the same bits, and neither may touch the padding columns or rows past the tail
    p = _problem(O, I, T, "bf16", 0.2, 8100 + O + I + T)
    L = make_layer(p)
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    outs = []
    for mode in ("1", "0"):
        monkeypatch.setenv("MST_TC_TMA_OUT", mode)
        Y = torch.full((T + 3, O + 8), float("nan"), dtype=torch.bfloat16, device=dev())
        dX = torch.full((T + 3, I + 8), float("nan"), dtype=torch.bfloat16, device=dev())
        G = torch.full((O + 2, I + 4), float("nan"), dtype=torch.float32, device=dev())
        mst.mst_spmm_fwd(L.handle, X, I, T, Y, O + 8)
        mst.mst_spmm_bwd_x(L.handle, dY, O, T, dX, I + 8)
        mst.mst_dense_grad(dY, O, X, I, T, O, I, mst.MST_BF16, G)     # G is the first O*I elements of the buffer
        torch.cuda.synchronize()
        assert torch.isnan(Y[:, O:]).all() and torch.isnan(Y[T:]).all() and not torch.isnan(Y[:T, :O]).any()
        assert torch.isnan(dX[:, I:]).all() and torch.isnan(dX[T:]).all() and not torch.isnan(dX[:T, :I]).any()
        Gflat = G.view(-1)[: O * I]
        assert not torch.isnan(Gflat).any() and torch.isnan(G.view(-1)[O * I:]).all()
        outs.append((Y[:T, :O].clone(), dX[:T, :I].clone(), Gflat.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    Wm = np.where(p.mask == 1, p.W, np.float32(0))
    assert rel_err(host(outs[0][0]), oracle.fwd(p.X, Wm, p.mask)) <= TOL["bf16"]
    assert rel_err(host(outs[0][2]).reshape(O, I), oracle.dense_grad(p.dY, p.X)) <= 1e-5
    assert mst.mst_device_error_flags() == 0
    L.close()


def test_csc_view_is_rebuilt_on_demand_after_an_update():
    # the fused update leaves the CSC view stale for layers whose input gradient runs on the tensor path; the
    # CUDA-core input gradient, the CSC export and the structure check rebuild it when they need it
    p = _problem(256, 320, 200, "bf16", 0.2, 9400)
    L = make_layer(p)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    G = oracle.dense_grad(p.dY, p.X).astype(np.float32)
    Wn, Mn = _update_both(L, p, W, p.mask.copy(), G, 0.3, -1, 0.25, 5, 0)      # ends with validate
    st = mst.mst_topology_update(L.handle, 0.2, -1, 0.5, 5, 1, False, torch.from_numpy(G).to(dev()))   # stale again
    n_prune, _, n_rand, n_grad = oracle.mg_counts(0.2, int(Mn.sum()), -1, Mn.size, 0.5)
    Wn, Mn, *_ = oracle.mg_update(Wn, Mn, G, n_prune, n_grad, n_rand, 5, 1, p.layer_id)
    dXr = oracle.bwd_x(p.dY, Wn, Mn)
    dY = to_dev(p, "dY")
    for path in (mst.MST_PATH_TENSOR_CORE, mst.MST_PATH_CUDA_CORE):
        L.set_path(path)
        dX = torch.full((p.tokens, 320), float("nan"), dtype=torch.bfloat16, device=dev())
        L.bwd_x(dY, dX, p.tokens)
        torch.cuda.synchronize()
        assert rel_err(host(dX), dXr) <= TOL["bf16"], path
    cp, ri, pm = export_csc(L)
    rp, ci, _ = export_csr(L, "bf16")
    rows = np.repeat(np.arange(256), np.diff(rp))
    order = np.lexsort((rows, ci))                   # CSC order: by column, then row
    np.testing.assert_array_equal(ri, rows[order])
    np.testing.assert_array_equal(pm, order)
    np.testing.assert_array_equal(cp, np.concatenate([[0], np.cumsum(np.bincount(ci, minlength=320))]))
    L.close()


# ------------------------------------------------------------ value tracking, path query, launch counter
def test_value_tracking_reuses_and_refreshes_derived_operands():
    from cuda.bindings import runtime as cudart
    p = _problem(192, 256, 300, "bf16", 0.2, 4321)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    for path in (mst.MST_PATH_TENSOR_CORE, mst.MST_PATH_SPARSE_TC):
        L = make_layer(p)
        L.set_path(path)
        L.track_values(True)
        T, O, I = p.tokens, p.out_features, p.in_features
        X, dY = to_dev(p, "X"), to_dev(p, "dY")
        Y = torch.empty((T, O), dtype=torch.bfloat16, device=dev())
        dX = torch.empty((T, I), dtype=torch.bfloat16, device=dev())

        def run():
            L.fwd(X, Y, T); L.bwd_x(dY, dX, T)
            torch.cuda.synchronize()
            return host(Y), host(dX)
        n0 = mst.mst_launch_count()
        Y1, dX1 = run()
        n1 = mst.mst_launch_count()
        Y2, dX2 = run()                      # nothing changed: the derived operands are reused, fewer launches
        n2 = mst.mst_launch_count()
        assert n2 - n1 < n1 - n0
        np.testing.assert_array_equal(Y1.view(np.uint32), Y2.view(np.uint32))
        assert rel_err(Y1, oracle.fwd(p.X, W, p.mask)) <= TOL["bf16"]
        # an optimizer step in place (every value doubled: exact in bf16), announced to the library
        ptr, nnz = mst.mst_values(L.handle)
        v2 = (2.0 * oracle.to_csr(W, p.mask)[2]).astype(np.float32)
        bits = torch.from_numpy(mst_inputs.f32_to_bf16_bits(v2).view(np.int16)).to(dev())
        (err,) = cudart.cudaMemcpy(ptr, bits.data_ptr(), 2 * nnz, cudart.cudaMemcpyKind.cudaMemcpyDeviceToDevice)
        assert int(err) == 0
        L.values_changed()
        Y3, dX3 = run()
        assert rel_err(Y3, oracle.fwd(p.X, 2.0 * W, p.mask)) <= TOL["bf16"]
        assert rel_err(dX3, oracle.bwd_x(p.dY, 2.0 * W, p.mask)) <= TOL["bf16"]
        # a topology update announces itself
        G = oracle.dense_grad(p.dY, p.X).astype(np.float32)
        st = mst.mst_topology_update(L.handle, 0.3, -1, 0.25, 3, 0, False, torch.from_numpy(G).to(dev()))
        Wn, Mn, *_ = oracle.mg_update((2.0 * W).astype(np.float32), p.mask.copy(), G, st.n_prune, st.n_grad, st.n_rand, 3, 0,
                                      p.layer_id)
        Y4, dX4 = run()
        assert rel_err(Y4, oracle.fwd(p.X, Wn, Mn)) <= TOL["bf16"]
        assert rel_err(dX4, oracle.bwd_x(p.dY, Wn, Mn)) <= TOL["bf16"]
        L.close()


@pytest.mark.parametrize("track", [False, True])
def test_products_through_the_fully_dense_state_and_back(track):
    """A layer restored to every entry kept passes its values as the dense operand: products must follow in-place value
    changes there with and without value tracking, and the image must come back when the layer is sparsified again."""
    from cuda.bindings import runtime as cudart
    O, I, T = 264, 328, 520
    p = _problem(O, I, T, "bf16", 0.3, 8642)
    L = make_layer(p)                         # capacity = O*I
    L.set_path(mst.MST_PATH_TENSOR_CORE)
    L.track_values(track)
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    Y = torch.empty((T, O), dtype=torch.bfloat16, device=dev())
    dX = torch.empty((T, I), dtype=torch.bfloat16, device=dev())

    def check(W, M):
        dW = torch.empty((max(int(M.sum()), 1),), dtype=torch.float32, device=dev())
        L.fwd(X, Y, T); L.bwd_x(dY, dX, T); L.sddmm(dY, X, T, dW)
        torch.cuda.synchronize()
        rows, cols = np.nonzero(M)
        assert rel_err(host(Y), oracle.fwd(p.X, W, M)) <= TOL["bf16"]
        assert rel_err(host(dX), oracle.bwd_x(p.dY, W, M)) <= TOL["bf16"]
        assert rel_err(host(dW)[: len(rows)], oracle.dense_grad(p.dY, p.X)[rows, cols]) <= TOL["bf16"]

    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    M = p.mask.copy()
    check(W, M)
    rng = np.random.default_rng(3)
    G = rng.standard_normal((O, I)).astype(np.float32)
    W, M = _update_both(L, p, W, M, G, 0.1, O * I, 0.25, 9, 0)           # restored: every entry kept, grown ones zero
    assert int(M.sum()) == O * I
    check(W, M)
    # an optimizer step in the dense state: new values written in place
    W = mst_inputs.bf16_bits_to_f32(mst_inputs.f32_to_bf16_bits((0.02 * rng.standard_normal((O, I))).astype(np.float32)))
    ptr, nnz = mst.mst_values(L.handle)
    assert nnz == O * I
    bits = torch.from_numpy(mst_inputs.f32_to_bf16_bits(W).view(np.int16)).to(dev())      # CSR order of a full matrix = row-major
    (err,) = cudart.cudaMemcpy(ptr, bits.data_ptr(), 2 * nnz, cudart.cudaMemcpyKind.cudaMemcpyDeviceToDevice)
    assert int(err) == 0
    L.values_changed()
    check(W, M)
    W, M = _update_both(L, p, W, M, G, 0.2, int(0.4 * O * I), 0.25, 9, 1)  # sparsified again
    check(W, M)
    assert mst.mst_device_error_flags() == 0
    L.close()


def test_path_in_use_reports_the_resolved_path():
    p = _problem(64, 64, 8, "bf16", 0.1, 1)
    L = make_layer(p)
    assert L.path_in_use() == mst.MST_PATH_TENSOR_CORE           # AUTO on an aligned bf16 layer
    L.set_path(mst.MST_PATH_CUDA_CORE)
    assert L.path_in_use() == mst.MST_PATH_CUDA_CORE
    L.set_path(mst.MST_PATH_SPARSE_TC)
    assert L.path_in_use() == mst.MST_PATH_SPARSE_TC
    L.close()
    q = _problem(64, 64, 8, "f32", 0.1, 1)
    L = make_layer(q)
    assert L.path_in_use() == mst.MST_PATH_CUDA_CORE             # fp32 layers never leave the CUDA cores
    L.close()


# ------------------------------------------------------------ several layers updated in one call
@pytest.mark.parametrize("shared_launch", ["0", "1"])
def test_update_many_is_bit_identical_to_single_updates(shared_launch, monkeypatch):
    monkeypatch.setenv("MST_UPDATE_BATCH", shared_launch)      # read by the library at every call
    shapes = [(96, 160, "bf16", 0.2), (130, 257, "bf16", 0.1), (64, 64, "f32", 0.3), (200, 96, "bf16", 0.05),
              (300, 200, "bf16", 0.5)]
    probs = [_problem(O, I, 4, dt, d, 700 + k) for k, (O, I, dt, d) in enumerate(shapes)]
    rng = np.random.default_rng(12)
    Gs = [np.round(rng.normal(size=(p.out_features, p.in_features)) * 4).astype(np.float32) / 4 for p in probs]   # many equal |g|
    Gd = [torch.from_numpy(g).to(dev()) for g in Gs]
    A = [make_layer(p) for p in probs]      # updated one by one
    Bm = [make_layer(p) for p in probs]     # updated together
    # growth, shrinkage, pure pruning (ties among the zeros grown before), R = 0 and R = 1
    plan = [(0.3, None, 0.25), (0.2, 0.9, 0.0), (0.1, 1.2, 1.0), (0.5, None, 0.5), (0.0, 0.5, 0.25), (0.3, None, 0.25)]
    for step, (zeta, scale, R) in enumerate(plan):
        targets = [-1 if scale is None else min(p.mask.size, max(0, int(L.nnz * scale))) for p, L in zip(probs, A)]
        for L, t, g in zip(A, targets, Gd):
            mst.mst_topology_update(L.handle, zeta, t, R, 21, step, False, g)
        rules = [mst.RegrowRule(int(t), float(R), 21, step, 0, 0.0) for t in targets]
        stats = mst.mst_topology_update_many([L.handle for L in Bm], [zeta] * len(Bm), rules, Gd)
        for p, La, Lb, st in zip(probs, A, Bm, stats):
            assert La.nnz == Lb.nnz == st.nnz_after
            for x, y in zip(export_csr(La, p.dtype), export_csr(Lb, p.dtype)):
                np.testing.assert_array_equal(x, y)
            Lb.validate()
    assert mst.mst_device_error_flags() == 0
    for L in A + Bm:
        L.close()


def test_update_many_checks_every_layer_first():
    p = _problem(64, 96, 4, "bf16", 0.2, 31)
    L1, L2 = make_layer(p), make_layer(p)
    n1, n2 = L1.nnz, L2.nnz
    G = torch.zeros((64, 96), dtype=torch.float32, device=dev())
    rules = [mst.RegrowRule(-1, 0.25, 1, 0, 0, 0.0), mst.RegrowRule(64 * 96 + 1, 0.25, 1, 0, 0, 0.0)]   # second: infeasible target
    with pytest.raises(mst.MstError) as e:
        mst.mst_topology_update_many([L1.handle, L2.handle], [0.3, 0.3], rules, [G, G])
    assert e.value.status == 5
    before = export_csr(L1, "bf16")
    assert (L1.nnz, L2.nnz) == (n1, n2)
    with pytest.raises(mst.MstError):            # the same layer twice
        mst.mst_topology_update_many([L1.handle, L1.handle], [0.3, 0.3], [rules[0], rules[0]], [G, G])
    for x, y in zip(before, export_csr(L1, "bf16")):
        np.testing.assert_array_equal(x, y)
    L1.close(); L2.close()
