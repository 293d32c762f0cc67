"""Full-size workloads (the five configurations) through the C ABI in the launch configuration the benchmark uses.

At these sizes the oracle computes sampled outputs one by one (fwd_at / bwd_x_at / grad_at); the topology update is
compared bit-exactly on whole layers (the oracle's sort of a few million keys takes about a second).
"""
import numpy as np
import pytest

import mst_inputs
import oracle

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import TOL, dev, export_csr, host, make_layer, mdtype, rel_err, tdtype, to_dev, value_bits

N_TOKENS = 64      # complete tokens checked per product (every output feature of each)
N_ROWS = 48        # complete weight rows checked for the weight gradient and the dense gradient


def _edge_indices(n, count, rng):
    """`count` indices in [0, n): the two sides of every 128 / 240 / 256 boundary of a few tiles spread over the
    range (first and last tile included: tile edges, the ragged tail and the last wave are where a tiling mistake
    shows), the rest random."""
    picks = {0, n - 1}
    for tile in (128, 240, 256):
        nt = (n + tile - 1) // tile
        for k in sorted({1, nt // 3, nt // 2, (2 * nt) // 3, nt - 1}):
            for v in (k * tile - 1, k * tile):
                if 0 <= v < n:
                    picks.add(v)
    picks = sorted(picks)
    if len(picks) > count:
        keep = rng.choice(len(picks), count, replace=False)
        picks = sorted(picks[j] for j in keep)
    rest = count - len(picks)
    if rest > 0:
        extra = rng.choice(n, min(n, rest), replace=False)
        picks = sorted(set(picks) | set(int(v) for v in extra))
    return np.asarray(picks, dtype=np.int64)


def _sampled_products_ok(p, L, rng, mask=None, Wm=None):
    """fwd / bwd_x / sddmm / dense_grad at full size.  Checked on whole slices instead of scattered points, so that a
    fault confined to one tile, one K-range split or the last ragged wave cannot slip through: every output of
    N_TOKENS complete tokens (forward and input gradient) and every entry of N_ROWS complete weight rows (weight
    gradient on the mask and dense gradient), tile edges included."""
    T, O, I = p.tokens, p.out_features, p.in_features
    mask = p.mask if mask is None else mask
    Wm = np.where(mask == 1, p.W, np.float32(0)) if Wm is None else Wm
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    Y = torch.empty((T, O), dtype=tdtype(p), device=dev())
    dX = torch.empty((T, I), dtype=tdtype(p), device=dev())
    nnz = L.nnz
    dW = torch.full((max(nnz, 1),), float("nan"), dtype=torch.float32, device=dev())
    G = torch.empty((O, I), dtype=torch.float32, device=dev())
    L.fwd(X, Y, T); L.bwd_x(dY, dX, T); L.sddmm(dY, X, T, dW); L.dense_grad(dY, X, T, G)
    torch.cuda.synchronize()
    tol = TOL[p.dtype]
    ts = _edge_indices(T, N_TOKENS, rng)
    tsd = torch.from_numpy(ts).to(dev())
    Yr = oracle.fwd(np.ascontiguousarray(p.X[ts]), Wm, mask)
    dXr = oracle.bwd_x(np.ascontiguousarray(p.dY[ts]), Wm, mask)
    # the scale of the tolerance is the largest reference value of the checked slice (a stricter bar than the
    # whole output's maximum)
    assert rel_err(host(Y[tsd]), Yr) <= tol
    assert rel_err(host(dX[tsd]), dXr) <= tol
    os_ = _edge_indices(O, N_ROWS, rng)
    Gr = oracle.dense_grad(np.ascontiguousarray(p.dY[:, os_]), p.X)            # [len(os_) x I], fp64
    assert rel_err(host(G[torch.from_numpy(os_).to(dev())]), Gr) <= tol
    if nnz:
        rp = np.concatenate([[0], np.cumsum(mask.sum(1, dtype=np.int64))])
        dWh = host(dW)
        assert not np.isnan(dWh[:nnz]).any()
        got = np.concatenate([dWh[rp[o]:rp[o + 1]] for o in os_])
        ref = np.concatenate([Gr[j, np.nonzero(mask[o])[0]] for j, o in enumerate(os_)])
        if ref.size:
            assert rel_err(got, ref) <= tol
    return G


def _update_and_compare(L, p, W, M, G_host, zeta, R, seed, step):
    O, I = M.shape
    Gd = torch.from_numpy(G_host).to(dev())
    st = mst.mst_topology_update(L.handle, zeta, -1, R, seed, step, False, Gd)
    n_prune, _, n_rand, n_grad = oracle.mg_counts(zeta, int(M.sum()), -1, O * I, R)
    assert (st.n_prune, st.n_rand, st.n_grad) == (n_prune, n_rand, n_grad)
    Wn, Mn, *_ = oracle.mg_update(W, M, G_host, n_prune, n_grad, n_rand, seed, step, p.layer_id)
    rp, ci, vb = export_csr(L, p.dtype)
    rp_r, ci_r, v_r = oracle.to_csr(Wn, Mn)
    np.testing.assert_array_equal(rp, rp_r)
    np.testing.assert_array_equal(ci, ci_r)
    np.testing.assert_array_equal(vb, value_bits(v_r, p.dtype))
    assert st.nnz_after == int(M.sum())
    return Wn, Mn


def test_config1_fp32_single_layer_full_check():
    (p,) = mst_inputs.config1()
    L = make_layer(p)
    assert L.nnz == 589824
    T, O, I = p.tokens, p.out_features, p.in_features
    X, dY = to_dev(p, "X"), to_dev(p, "dY")
    Y = torch.empty((T, O), device=dev()); dX = torch.empty((T, I), device=dev())
    dW = torch.empty((L.nnz,), device=dev()); G = torch.empty((O, I), device=dev())
    L.fwd(X, Y, T); L.bwd_x(dY, dX, T); L.sddmm(dY, X, T, dW); L.dense_grad(dY, X, T, G)
    torch.cuda.synchronize()
    Wm = np.where(p.mask == 1, p.W, np.float32(0))
    Gr = oracle.dense_grad(p.dY, p.X)
    rows, cols = np.nonzero(p.mask)
    assert rel_err(host(Y), oracle.fwd(p.X, Wm, p.mask)) <= 1e-5
    assert rel_err(host(dX), oracle.bwd_x(p.dY, Wm, p.mask)) <= 1e-5
    assert rel_err(host(dW), Gr[rows, cols]) <= 1e-5
    assert rel_err(host(G), Gr) <= 1e-5
    # one update, zeta = 0.3, R = 0.25, on the oracle's dense gradient rounded to fp32
    _update_and_compare(L, p, Wm.astype(np.float32), p.mask.copy(), Gr.astype(np.float32), 0.3, 0.25, 0x4D5354, 0)
    L.validate()
    L.close()


def test_config2_gpt2_small_block_bf16():
    rng = np.random.default_rng(2)
    for p in mst_inputs.config2():
        L = make_layer(p)
        assert L.nnz == mst_inputs.exact_nnz(p.out_features, p.in_features, 0.25)
        _sampled_products_ok(p, L, rng)
        L.close()
    assert mst.mst_device_error_flags() == 0


@pytest.mark.parametrize("block", list(range(12)))
def test_config3_zipf_rows_update_every_step(block):
    rng = np.random.default_rng(3 + block)
    for p in mst_inputs.config3(blocks=1, first_block=block):
        L = make_layer(p)
        d = p.nnz / p.mask.size
        assert 0.03 - 1e-6 <= d <= 0.10 + 1e-6 and int(p.mask.sum(1).max()) == p.in_features   # saturated heavy rows
        G = _sampled_products_ok(p, L, rng)
        W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
        M = p.mask.copy()
        Gh = host(G)
        for step in range(3 if block in (0, 7) else 2):   # from the second step on the just-grown zeros tie at |w| = 0
            W, M = _update_and_compare(L, p, W, M, Gh, 0.1, 0.25, 0x4D5354 + 3, step)
        L.validate()
        # the products still agree on the evolved structure
        _sampled_products_ok(p, L, rng, mask=M, Wm=W)
        L.close()
    assert mst.mst_device_error_flags() == 0


@pytest.mark.parametrize("block", [11, 23])
def test_config4_other_blocks_products(block):
    # the 24 blocks differ only in their seeds; the middle and the last one are checked on the products alone
    rng = np.random.default_rng(40 + block)
    for p in mst_inputs.config4(blocks=1, first_block=block):
        L = make_layer(p)
        _sampled_products_ok(p, L, rng)
        L.close()
    assert mst.mst_device_error_flags() == 0


def test_config4_gpt2_medium_block_with_regrowth():
    rng = np.random.default_rng(4)
    for p in mst_inputs.config4(blocks=1):
        L = make_layer(p)
        G = _sampled_products_ok(p, L, rng)
        W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
        Gh = host(G)
        for R in (0.0, 0.25):          # pure gradient growth, then the mixed rule, each from the packed state
            L2 = make_layer(p)
            _update_and_compare(L2, p, W, p.mask.copy(), Gh, 0.3, R, 0x4D5354 + 4, 0)
            L2.close()
        L.close()
    assert mst.mst_device_error_flags() == 0


def test_config5_density_sweep_gpt2_large_shapes():
    rng = np.random.default_rng(5)
    base = mst_inputs.config5(1.0)
    for p in base:
        O, I = p.out_features, p.in_features
        for d in mst_inputs.CONFIG5_DENSITIES:
            nnz = mst_inputs.exact_nnz(O, I, d)
            mask = np.ones((O, I), dtype=np.uint8) if d == 1.0 else mst_inputs.uniform_mask(O, I, nnz, 50 + int(d * 100), p.layer_id)
            L = mst.Layer(p.layer_id, O, I, mst.MST_BF16)
            L.pack(to_dev(p, "W"), torch.from_numpy(mask).to(dev()))
            assert L.nnz == nnz
            _sampled_products_ok(p, L, rng, mask=mask)
            L.close()
    assert mst.mst_device_error_flags() == 0


def test_lm_head_shape_large_out_features():
    # the output layer of GPT-2 small (768 -> 50304) is sparsified too in the paper's FLOP model: a very wide O
    rng = np.random.default_rng(6)
    O, I, T = 50304, 768, 2048
    p = mst_inputs.uniform_layer("lm_head", 0, O, I, T, "bf16", 0.1, 4242)
    L = make_layer(p)
    assert L.nnz == mst_inputs.exact_nnz(O, I, 0.1)
    L.validate()
    G = _sampled_products_ok(p, L, rng)
    W = np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32)
    _update_and_compare(L, p, W, p.mask.copy(), host(G), 0.3, 0.25, 11, 0)
    L.close()
    assert mst.mst_device_error_flags() == 0


@pytest.mark.parametrize("shared_launch", ["0", "1"])
def test_config3_block_updated_in_one_call(shared_launch, monkeypatch):
    monkeypatch.setenv("MST_UPDATE_BATCH", shared_launch)
    # the four layers of an ultra-sparse block (Zipf rows) updated together, every step, against the oracle
    probs = mst_inputs.config3(blocks=1, first_block=3)
    layers = [make_layer(p) for p in probs]
    rng = np.random.default_rng(33)
    Ws = [np.where(p.mask == 1, p.W, np.float32(0)).astype(np.float32) for p in probs]
    Ms = [p.mask.copy() for p in probs]
    Gh = [rng.normal(size=p.mask.shape).astype(np.float32) for p in probs]
    Gd = [torch.from_numpy(g).to(dev()) for g in Gh]
    for step in range(3):
        rules = [mst.RegrowRule(-1, 0.25, 77, step, 0, 0.0) for _ in probs]
        stats = mst.mst_topology_update_many([L.handle for L in layers], [0.1] * 4, rules, Gd)
        for j, (p, L, st) in enumerate(zip(probs, layers, stats)):
            n_prune, _, n_rand, n_grad = oracle.mg_counts(0.1, int(Ms[j].sum()), -1, Ms[j].size, 0.25)
            assert (st.n_prune, st.n_rand, st.n_grad) == (n_prune, n_rand, n_grad)
            Ws[j], Ms[j], *_ = oracle.mg_update(Ws[j], Ms[j], Gh[j], n_prune, n_grad, n_rand, 77, step, p.layer_id)
            rp, ci, vb = export_csr(L, p.dtype)
            rp_r, ci_r, v_r = oracle.to_csr(Ws[j], Ms[j])
            np.testing.assert_array_equal(rp, rp_r)
            np.testing.assert_array_equal(ci, ci_r)
            np.testing.assert_array_equal(vb, value_bits(v_r, p.dtype))
    for L in layers:
        L.validate()
        L.close()
    assert mst.mst_device_error_flags() == 0
