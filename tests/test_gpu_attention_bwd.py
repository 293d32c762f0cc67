"""Strided sparse attention backward vs the CPU checker (needs a GPU)."""
import numpy as np
import pytest

import mst_inputs
from oracle import attention as oatt

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import dev, host, rel_err


def _run(B, n, H, stride, seed, pad=0, std=1.0):
    d, C = 64, H * 64
    p = mst_inputs.attention_problem(B, n, H, d, seed=seed, std=std)
    g = mst_inputs.attention_problem(B, n, H, d, seed=seed + 1, std=1.0)     # upstream gradient: first C columns
    ld = 3 * C + pad
    qkv = torch.full((B * n, ld), float("nan"), dtype=torch.bfloat16, device=dev())
    qkv[:, : 3 * C] = torch.from_numpy(p.qkv_bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    dO_bits = np.ascontiguousarray(g.qkv_bits[:, :C])
    dO = torch.from_numpy(dO_bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    # forward output and log-sum-exp from the checker (rounded to the stored precisions), so that the backward kernels
    # are tested on their own, also at strides the forward kernel does not cover
    Q, K, V = p.split()
    out_r, lse_r = oatt.strided_attention(Q, K, V, stride)
    out_bits = mst_inputs.f32_to_bf16_bits(np.ascontiguousarray(out_r.transpose(0, 2, 1, 3).reshape(B * n, C)).astype(np.float32))
    out = torch.from_numpy(out_bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    lse = torch.from_numpy(lse_r.astype(np.float32)).to(dev())
    base = qkv.data_ptr()
    dqkv = torch.full((B * n, ld), float("nan"), dtype=torch.bfloat16, device=dev())
    gb = dqkv.data_ptr()
    mst.mst_strided_attention_bwd(base, base + 2 * C, base + 4 * C, ld, out, C, dO, C, lse, B, n, H, d, stride,
                                  gb, gb + 2 * C, gb + 4 * C, ld)
    torch.cuda.synchronize()
    dOr = mst_inputs.bf16_bits_to_f32(dO_bits).reshape(B, n, H, d).transpose(0, 2, 1, 3)
    dQ, dK, dV = oatt.strided_attention_bwd(Q, K, V, dOr, stride)
    got = host(dqkv)[:, : 3 * C].reshape(B, n, 3, H, d).transpose(2, 0, 3, 1, 4)     # [3, B, H, n, d]
    return got, (dQ, dK, dV), dqkv


@pytest.mark.parametrize("B,n,H,stride,pad,std", [
    (1, 256, 1, 128, 0, 1.0),       # one strided key per late query, no far keys
    (2, 512, 3, 128, 0, 1.0),       # far keys i - 2l, i - 3l; two sequences
    (1, 1024, 2, 256, 8, 1.0),      # the paper's stride at n = 1024, padded leading dimension
    (1, 512, 2, 512, 0, 1.0),       # stride = n: plain causal attention
    (1, 384, 2, 64, 0, 2.0),        # smallest stride, peaked scores
    (1, 1024, 1, 64, 0, 1.0),       # up to fourteen strided positions beyond the window: many diagonal-only tiles
    (1, 768, 2, 192, 8, 1.0)])      # a stride that is not a power of two
def test_attention_bwd_matches_oracle(B, n, H, stride, pad, std):
    got, ref, _ = _run(B, n, H, stride, 900 + n + stride, pad, std)
    for a, b, name in zip(got, ref, ("dQ", "dK", "dV")):
        assert rel_err(a, b) <= 2e-2, name
    assert mst.mst_device_error_flags() == 0


def test_attention_bwd_after_the_forward_kernel():
    # the forward kernel's own output and log-sum-exp feed the backward kernels
    B, n, H, stride, d = 1, 512, 2, 128, 64
    C = H * d
    p = mst_inputs.attention_problem(B, n, H, d, seed=77)
    g = mst_inputs.attention_problem(B, n, H, d, seed=78)
    qkv = torch.from_numpy(p.qkv_bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    dO_bits = np.ascontiguousarray(g.qkv_bits[:, :C])
    dO = torch.from_numpy(dO_bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    out = torch.empty((B * n, C), dtype=torch.bfloat16, device=dev())
    lse = torch.empty((B, H, n), dtype=torch.float32, device=dev())
    base = qkv.data_ptr()
    mst.mst_strided_attention_fwd(base, base + 2 * C, base + 4 * C, 3 * C, B, n, H, d, stride, out, C, lse)
    dqkv = torch.empty((B * n, 3 * C), dtype=torch.bfloat16, device=dev())
    gb = dqkv.data_ptr()
    mst.mst_strided_attention_bwd(base, base + 2 * C, base + 4 * C, 3 * C, out, C, dO, C, lse, B, n, H, d, stride,
                                  gb, gb + 2 * C, gb + 4 * C, 3 * C)
    torch.cuda.synchronize()
    Q, K, V = p.split()
    dOr = mst_inputs.bf16_bits_to_f32(dO_bits).reshape(B, n, H, d).transpose(0, 2, 1, 3)
    ref = oatt.strided_attention_bwd(Q, K, V, dOr, stride)
    got = host(dqkv).reshape(B, n, 3, H, d).transpose(2, 0, 3, 1, 4)
    for a, b, name in zip(got, ref, ("dQ", "dK", "dV")):
        assert rel_err(a, b) <= 2e-2, name


def test_attention_bwd_is_deterministic_and_checks_arguments():
    got1, _, _ = _run(1, 512, 2, 128, 5)
    got2, _, _ = _run(1, 512, 2, 128, 5)
    np.testing.assert_array_equal(got1.view(np.uint32), got2.view(np.uint32))
    x = torch.zeros((256, 192), dtype=torch.bfloat16, device=dev())
    lse = torch.zeros((1, 1, 256), dtype=torch.float32, device=dev())
    with pytest.raises(mst.MstError) as e:      # head_dim 32 is not supported
        mst.mst_strided_attention_bwd(x, x, x, 192, x, 192, x, 192, lse, 1, 256, 1, 32, 128, x, x, x, 192)
    assert e.value.status == 2
    with pytest.raises(mst.MstError) as e:      # sequence length not a multiple of 64
        mst.mst_strided_attention_bwd(x, x, x, 192, x, 192, x, 192, lse, 1, 200, 1, 64, 128, x, x, x, 192)
    assert e.value.status == 2


def test_attention_bwd_random_shapes():
    # sequence lengths and strides drawn at random (multiples of 64), one call after the other in one process
    rng = np.random.default_rng(21)
    for case in range(14):
        n = 64 * int(rng.integers(1, 13))
        stride = 64 * int(rng.integers(1, n // 64 + 1))
        B, H = int(rng.integers(1, 3)), int(rng.integers(1, 4))
        pad = int(rng.choice([0, 8]))
        got, ref, _ = _run(B, n, H, stride, 1300 + case, pad, float(rng.choice([0.5, 1.0, 1.5])))
        for a, b, name in zip(got, ref, ("dQ", "dK", "dV")):
            assert rel_err(a, b) <= 2e-2, (case, name, B, n, H, stride, pad)
