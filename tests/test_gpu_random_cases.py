"""Seeded random cases through the C ABI vs the CPU checker (needs a GPU): shapes, densities, dtypes, kernel families
and update rules drawn at random, many small layers one after the other in one process -- what the fixed cases of the
other files do not cover is the ORDER of calls (function attributes, cached operands and scratch left by one layer
must not leak into the next)."""
import numpy as np
import pytest

import mst_inputs
import oracle

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import TOL, dev, export_csr, host, make_layer, mdtype, rel_err, tdtype, to_dev, value_bits


@pytest.mark.parametrize("seed", [1, 2])
def test_random_updates_are_bit_exact(seed):
    rng = np.random.default_rng(seed)
    for case in range(60):
        O, I = int(rng.integers(1, 260)), int(rng.integers(1, 420))
        if rng.random() < 0.15:
            O, I = int(rng.integers(300, 900)), int(rng.integers(256, 1100))
        dtype = "bf16" if rng.random() < 0.6 else "f32"
        density = float(rng.choice([0.0, 0.02, 0.1, 0.3, 0.7, 1.0, rng.random()]))
        zipf = rng.random() < 0.2 and density > 0
        p = (mst_inputs.zipf_layer if zipf else mst_inputs.uniform_layer)("t", case % 7, O, I, 4, dtype, density, 9000 + case)
        L = make_layer(p)
        W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
        M = p.mask.copy()
        allow = bool(rng.random() < 0.2)
        lam = float(rng.choice([0.0, 0.0, 0.5]))
        for step in range(3):
            zeta = float(rng.choice([0.0, 0.1, 0.3, 0.5, 1.0, rng.random()]))
            R = float(rng.choice([0.0, 0.25, 0.5, 1.0, rng.random()]))
            tgt = -1 if rng.random() < 0.5 else int(rng.integers(0, O * I + 1))
            G = rng.standard_normal((O, I)).astype(np.float32)
            if rng.random() < 0.4:      # few distinct magnitudes: ties in the gradient selection
                G = rng.choice(np.array([0.5, -0.5, 0.25, -1.0, 0.0], dtype=np.float32), size=(O, I))
            c = oracle.mg_counts(zeta, int(M.sum()), tgt, O * I, R)
            st = mst.mst_topology_update(L.handle, zeta, tgt, R, 77, step, allow, torch.from_numpy(G).to(dev()),
                                         prune_grad_weight=lam)
            assert (st.n_prune, st.n_rand, st.n_grad) == (c[0], c[2], c[3])
            W, M, *_ = oracle.mg_update(W, M, G, c[0], c[3], c[2], 77, step, p.layer_id, allow, lam)
            rp, ci, vb = export_csr(L, dtype)
            rp_r, ci_r, v_r = oracle.to_csr(W, M)
            what = (case, step, O, I, dtype, density, zeta, R, tgt, allow, lam)
            assert np.array_equal(rp, rp_r) and np.array_equal(ci, ci_r), what
            assert np.array_equal(vb, value_bits(v_r, dtype)), what
        L.close()


@pytest.mark.parametrize("seed", [3])
def test_random_products_on_every_kernel_family(seed):
    rng = np.random.default_rng(seed)
    paths = [mst.MST_PATH_AUTO, mst.MST_PATH_CUDA_CORE, mst.MST_PATH_TENSOR_CORE, mst.MST_PATH_SPARSE_TC]
    for case in range(60):
        O, I, T = int(rng.integers(1, 420)), int(rng.integers(1, 520)), int(rng.integers(1, 700))
        if rng.random() < 0.5:
            O, I = (O + 7) // 8 * 8, (I + 7) // 8 * 8      # operands the tensor paths accept
        dtype = "bf16" if rng.random() < 0.7 else "f32"
        density = float(rng.choice([0.0, 0.02, 0.1, 0.25, 0.6, 1.0, rng.random()]))
        zipf = rng.random() < 0.25 and density > 0
        p = (mst_inputs.zipf_layer if zipf else mst_inputs.uniform_layer)("t", case % 5, O, I, T, dtype, density, 7000 + case)
        L = make_layer(p)
        path = int(rng.choice(paths))
        L.set_path(path)
        padx, pady = int(rng.choice([0, 8, 16])), int(rng.choice([0, 8]))
        ldx, ldy = I + padx, O + pady
        X, dY = to_dev(p, "X", ldx if padx else None), to_dev(p, "dY", ldy if pady else None)
        Y = torch.full((T, ldy), float("nan"), dtype=tdtype(p), device=dev())
        dX = torch.full((T, ldx), float("nan"), dtype=tdtype(p), device=dev())
        dW = torch.full((max(p.nnz, 1),), float("nan"), dtype=torch.float32, device=dev())
        G = torch.full((O, I), float("nan"), dtype=torch.float32, device=dev())
        mst.mst_spmm_fwd(L.handle, X, ldx, T, Y, ldy)
        mst.mst_spmm_bwd_x(L.handle, dY, ldy, T, dX, ldx)
        mst.mst_sddmm_dw(L.handle, dY, ldy, X, ldx, T, dW)
        mst.mst_dense_grad(dY, ldy, X, ldx, T, O, I, mdtype(p), G)
        torch.cuda.synchronize()
        Wm = np.where(p.mask == 1, p.W, np.float32(0))
        Gr = oracle.dense_grad(p.dY, p.X)
        what = (case, O, I, T, dtype, density, path, padx, pady)
        assert rel_err(host(Y)[:, :O], oracle.fwd(p.X, Wm, p.mask)) <= TOL[dtype], what
        assert rel_err(host(dX)[:, :I], oracle.bwd_x(p.dY, Wm, p.mask)) <= TOL[dtype], what
        assert rel_err(host(G), Gr) <= TOL[dtype], what
        if p.nnz:
            rows, cols = np.nonzero(p.mask)
            assert rel_err(host(dW)[: p.nnz], Gr[rows, cols]) <= TOL[dtype], what
        assert mst.mst_device_error_flags() == 0, what
        L.close()


def test_random_sequences_of_calls_on_one_layer():
    # products on changing kernel families, updates, in-place value changes and value tracking in random order on
    # the same layer: cached operands (dense image, compressed 2:4 operand and its places, CSC view, longest row) must
    # follow every change
    from cuda.bindings import runtime as cudart
    rng = np.random.default_rng(8)
    paths = [mst.MST_PATH_AUTO, mst.MST_PATH_CUDA_CORE, mst.MST_PATH_TENSOR_CORE, mst.MST_PATH_SPARSE_TC]
    for case in range(24):
        O, I, T = 8 * int(rng.integers(4, 60)), 8 * int(rng.integers(4, 70)), int(rng.integers(8, 400))
        dtype = "bf16" if rng.random() < 0.75 else "f32"
        density = float(rng.choice([0.03, 0.1, 0.25, 0.5]))
        zipf = rng.random() < 0.25
        p = (mst_inputs.zipf_layer if zipf else mst_inputs.uniform_layer)("t", case % 5, O, I, T, dtype, density, 11000 + case)
        L = make_layer(p)
        W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
        if dtype == "bf16":
            W = mst_inputs.bf16_bits_to_f32(mst_inputs.f32_to_bf16_bits(W))
        M = p.mask.copy()
        X, dY = to_dev(p, "X"), to_dev(p, "dY")
        track, log = False, []
        for op_i in range(12):
            op = str(rng.choice(["prod", "prod", "update", "path", "scale", "track"]))
            log.append(op)
            if op == "path":
                L.set_path(int(rng.choice(paths)))
            elif op == "track":
                track = not track
                L.track_values(track)
            elif op == "scale":          # an optimizer step in place: every stored value doubled (exact)
                ptr, nnz = mst.mst_values(L.handle)
                if nnz:
                    _, _, v = oracle.to_csr(W, M)
                    v2 = (2.0 * v).astype(np.float32)
                    src = (torch.from_numpy(mst_inputs.f32_to_bf16_bits(v2).view(np.int16)) if dtype == "bf16" else torch.from_numpy(v2)).to(dev())
                    torch.cuda.synchronize()
                    (err,) = cudart.cudaMemcpy(ptr, src.data_ptr(), (2 if dtype == "bf16" else 4) * nnz,
                                               cudart.cudaMemcpyKind.cudaMemcpyDeviceToDevice)
                    assert int(err) == 0
                    W = (2.0 * W).astype(np.float32)
                    if track:
                        L.values_changed()
            elif op == "update":
                zeta, R = float(rng.choice([0.1, 0.3, 0.5])), float(rng.choice([0.0, 0.25, 1.0]))
                tgt = -1 if rng.random() < 0.6 else int(rng.integers(1, O * I // 2))
                G = rng.standard_normal((O, I)).astype(np.float32)
                c = oracle.mg_counts(zeta, int(M.sum()), tgt, O * I, R)
                mst.mst_topology_update(L.handle, zeta, tgt, R, 5, op_i, False, torch.from_numpy(G).to(dev()),
                                        want_stats=bool(rng.random() < 0.5))
                W, M, *_ = oracle.mg_update(W, M, G, c[0], c[3], c[2], 5, op_i, p.layer_id, False, 0.0)
            else:
                nnz = int(M.sum())
                Y = torch.full((T, O), float("nan"), dtype=tdtype(p), device=dev())
                dX = torch.full((T, I), float("nan"), dtype=tdtype(p), device=dev())
                dW = torch.full((max(nnz, 1),), float("nan"), dtype=torch.float32, device=dev())
                L.fwd(X, Y, T)
                L.bwd_x(dY, dX, T)
                L.sddmm(dY, X, T, dW)
                torch.cuda.synchronize()
                what = (case, O, I, T, dtype, density, log)
                assert rel_err(host(Y), oracle.fwd(p.X, W, M)) <= TOL[dtype], what
                assert rel_err(host(dX), oracle.bwd_x(p.dY, W, M)) <= TOL[dtype], what
                if nnz:
                    rows, cols = np.nonzero(M)
                    assert rel_err(host(dW)[:nnz], oracle.dense_grad(p.dY, p.X)[rows, cols]) <= TOL[dtype], what
        rp, ci, vb = export_csr(L, dtype)
        rp_r, ci_r, v_r = oracle.to_csr(W, M)
        assert np.array_equal(rp, rp_r) and np.array_equal(ci, ci_r) and np.array_equal(vb, value_bits(v_r, dtype)), (case, log)
        assert mst.mst_device_error_flags() == 0, (case, log)
        L.close()
