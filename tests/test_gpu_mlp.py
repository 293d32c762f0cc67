"""fc1 -> GELU -> fc2 with the activation fused behind the products, through the C ABI, against the oracle.

Each call is checked on its own inputs: the second layer's forward takes the H the library produced (its bf16 bits,
widened exactly), and the derivative is taken at the stored pre-activation bits, so no error carries across calls.
"""
import numpy as np
import pytest

import mst_inputs
import oracle
from oracle import activation as act

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import TOL, dev, host, make_layer, rel_err, tdtype, to_dev


def _pre_activation(T, C, dtype, seed):
    y = mst_inputs.normal((T, C), 1.5, seed, 77)
    if dtype == "bf16":
        bits = mst_inputs.f32_to_bf16_bits(y)
        return mst_inputs.bf16_bits_to_f32(bits), torch.from_numpy(bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    return y, torch.from_numpy(y).to(dev())


def _padded(t, ld):
    buf = torch.full((t.shape[0], ld), float("nan"), dtype=t.dtype, device=t.device)
    buf[:, : t.shape[1]] = t
    return buf


@pytest.mark.parametrize("dtype,path", [("bf16", "tensor"), ("bf16", "cuda_core"), ("f32", "cuda_core")])
@pytest.mark.parametrize("T,d,hid", [(300, 200, 520), (129, 64, 264), (1, 40, 72)])
def test_mlp_pair_small(dtype, path, T, d, hid):
    m1 = mst_inputs.uniform_mask(hid, d, mst_inputs.exact_nnz(hid, d, 0.3), 901, 1)
    m2 = mst_inputs.uniform_mask(d, hid, mst_inputs.exact_nnz(d, hid, 0.3), 901, 2)
    p1 = mst_inputs.make_layer("fc1", 1, hid, d, T, dtype, m1, 901, w_std=0.25)
    p2 = mst_inputs.make_layer("fc2", 2, d, hid, T, dtype, m2, 901, w_std=0.05)
    L1, L2 = make_layer(p1), make_layer(p2)
    for L in (L1, L2):
        L.set_path(mst.MST_PATH_TENSOR_CORE if path == "tensor" else mst.MST_PATH_CUDA_CORE)
    tol = TOL[dtype]
    X = to_dev(p1, "X")
    H = torch.empty((T, hid), dtype=tdtype(p1), device=dev())
    Ypre = torch.empty((T, hid), dtype=tdtype(p1), device=dev())
    L1.fwd_gelu(X, H, T, Y_pre=Ypre)
    H_only = torch.empty_like(H)
    L1.fwd_gelu(X, H_only, T)                       # without the pre-activation output
    torch.cuda.synchronize()
    Y1 = oracle.fwd(p1.X, p1.W, p1.mask)
    assert np.abs(Y1).max() > 2.0                    # the inputs reach both tails of the activation
    assert rel_err(host(Ypre), Y1) <= tol
    assert rel_err(host(H), act.gelu(Y1)) <= tol
    if dtype == "bf16" and path == "cuda_core":
        # without a pre-activation buffer the CUDA-core route rounds the product to bf16 before the activation
        assert rel_err(host(H_only), act.gelu(Y1)) <= tol
    else:
        assert torch.equal(H_only, H)
    # second layer on the H just produced
    Y2 = torch.empty((T, d), dtype=tdtype(p1), device=dev())
    L2.fwd(H, Y2, T)
    torch.cuda.synchronize()
    assert rel_err(host(Y2), oracle.fwd(host(H), p2.W, p2.mask)) <= tol
    # backward through fc2 and the activation in one call, derivative at given pre-activation bits
    pre_host, pre_dev = _pre_activation(T, hid, dtype, 33)
    dY = to_dev(p2, "dY")
    dPre = torch.empty((T, hid), dtype=tdtype(p1), device=dev())
    L2.bwd_x_gelu(dY, pre_dev, dPre, T)
    torch.cuda.synchronize()
    ref = oracle.bwd_x(p2.dY, p2.W, p2.mask) * act.gelu_grad(pre_host)
    assert rel_err(host(dPre), ref) <= tol
    # padded leading dimensions (the ragged store paths) give the same bits
    ld = hid + 8 if dtype == "bf16" else hid + 3
    Hp = torch.full((T, ld), float("nan"), dtype=H.dtype, device=dev())
    Yp = torch.full((T, ld), float("nan"), dtype=H.dtype, device=dev())
    mst.mst_spmm_fwd_gelu(L1.handle, X, d, T, Yp, ld, Hp, ld)
    dPp = torch.full((T, ld), float("nan"), dtype=H.dtype, device=dev())
    mst.mst_spmm_bwd_x_gelu(L2.handle, dY, d, T, _padded(pre_dev, ld), ld, dPp, ld)
    torch.cuda.synchronize()
    assert torch.equal(Hp[:, :hid], H) and torch.equal(Yp[:, :hid], Ypre) and torch.equal(dPp[:, :hid], dPre)
    assert torch.isnan(Hp[:, hid:]).all() and torch.isnan(dPp[:, hid:]).all()
    L1.close(); L2.close()
    assert mst.mst_device_error_flags() == 0


def test_mlp_pair_argument_errors():
    p = mst_inputs.uniform_layer("fc1", 1, 64, 32, 16, "bf16", 0.5, 5)
    L = make_layer(p)
    X = to_dev(p, "X")
    H = torch.empty((16, 64), dtype=torch.bfloat16, device=dev())
    with pytest.raises(mst.MstError) as e:
        mst.mst_spmm_fwd_gelu(L.handle, X, 32, 16, None, 0, H, 63)
    assert e.value.status == 2            # MST_ERR_SHAPE
    with pytest.raises(mst.MstError) as e:
        mst.mst_spmm_fwd_gelu(L.handle, X, 32, 16, H, 8, H, 64)
    assert e.value.status == 2            # MST_ERR_SHAPE
    with pytest.raises(mst.MstError) as e:
        mst.mst_spmm_bwd_x_gelu(L.handle, H, 64, 16, None, 32, X, 32)
    assert e.value.status == 1      # MST_ERR_INVALID_ARG
    mst.mst_spmm_fwd_gelu(L.handle, X, 32, 0, None, 0, H, 64)      # no tokens: nothing to do
    L.close()


def test_mlp_pair_gpt2_small_full_size():
    rng = np.random.default_rng(8)
    ps = {p.name: p for p in mst_inputs.config2()}
    p1, p2 = ps["fc1"], ps["fc2"]
    T, d, hid = p1.tokens, p1.in_features, p1.out_features
    L1, L2 = make_layer(p1), make_layer(p2)
    X = to_dev(p1, "X")
    H = torch.empty((T, hid), dtype=torch.bfloat16, device=dev())
    Ypre = torch.empty_like(H)
    L1.fwd_gelu(X, H, T, Y_pre=Ypre)
    pre_host, pre_dev = _pre_activation(T, hid, "bf16", 34)
    dPre = torch.empty_like(H)
    L2.bwd_x_gelu(to_dev(p2, "dY"), pre_dev, dPre, T)
    torch.cuda.synchronize()
    n = 3000
    t = rng.integers(0, T, n); o = rng.integers(0, hid, n)
    ti, oi = torch.from_numpy(t).to(dev()), torch.from_numpy(o).to(dev())
    y = oracle.fwd_at(p1.X, p1.W, p1.mask, t, o)
    assert rel_err(host(Ypre[ti, oi]), y) <= TOL["bf16"]
    assert rel_err(host(H[ti, oi]), act.gelu(y)) <= TOL["bf16"]
    ref = oracle.bwd_x_at(p2.dY, p2.W, p2.mask, t, o) * act.gelu_grad(pre_host[t, o])
    assert rel_err(host(dPre[ti, oi]), ref) <= TOL["bf16"]
    L1.close(); L2.close()
    assert mst.mst_device_error_flags() == 0
