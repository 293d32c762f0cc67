"""Strided sparse self-attention through the C ABI against the oracle's plain definition."""
import numpy as np
import pytest

import mst_inputs
import oracle
from oracle import attention as att

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import TOL, dev, host, rel_err


def _run(p, stride, want_lse=True, pad=0):
    """Launch on the three column slices of the fused qkv activation; returns (out [B, H, n, d], lse [B, H, n])."""
    C = p.heads * p.head_dim
    ld = 3 * C + pad
    qkv = torch.full((p.batch * p.seq, ld), float("nan"), dtype=torch.bfloat16, device=dev())
    qkv[:, : 3 * C] = torch.from_numpy(p.qkv_bits.view(np.int16)).to(dev()).view(torch.bfloat16)
    out = torch.full((p.batch * p.seq, C + pad), float("nan"), dtype=torch.bfloat16, device=dev())
    lse = torch.full((p.batch, p.heads, p.seq), float("nan"), dtype=torch.float32, device=dev()) if want_lse else None
    base = qkv.data_ptr()
    mst.mst_strided_attention_fwd(base, base + 2 * C, base + 4 * C, ld, p.batch, p.seq, p.heads, p.head_dim, stride, out,
                                  C + pad, lse)
    torch.cuda.synchronize()
    assert mst.mst_device_error_flags() == 0
    if pad:
        assert torch.isnan(out[:, C:]).all()
    o = host(out[:, :C]).reshape(p.batch, p.seq, p.heads, p.head_dim).transpose(0, 2, 1, 3)
    return o, (host(lse) if want_lse else None)


@pytest.mark.parametrize("batch,seq,heads,stride,pad", [
    (2, 512, 3, 128, 0),       # strided positions up to i - 3l, two sequences (keys in front of a sequence start)
    (1, 1024, 2, 256, 0),      # the paper's setting: n = 1024, l = 256
    (3, 256, 2, 256, 8),       # stride = n: plain causal attention inside one window; padded leading dimensions
    (2, 128, 1, 128, 0),       # a single query block
    (1, 1024, 1, 128, 0),      # seven strided positions
    (1, 2048, 2, 256, 0)])     # the longest sequence the tensor-memory kernel takes for l = 256: six positions outside the tile
@pytest.mark.parametrize("kernel", ["warp", "tcgen05"])
def test_forward_matches_oracle(batch, seq, heads, stride, pad, kernel, monkeypatch):
    monkeypatch.setenv("MST_ATTN_FWD", kernel)
    _check_forward(batch, seq, heads, stride, pad)


@pytest.mark.parametrize("batch,seq,heads,stride,pad", [
    (1, 512, 2, 64, 0),        # stride of one tile: seven strided positions per half block
    (2, 384, 1, 192, 8),       # stride an odd multiple of 64: the two halves of a block reach back differently
    (1, 640, 2, 320, 0),
    (1, 1024, 1, 512, 0),      # window longer than a block's span
    (2, 256, 2, 1024, 0),      # stride beyond the sequence: plain causal attention
    (1, 4096, 1, 128, 0)])     # 31 strided positions
def test_forward_strides_of_the_warp_level_kernel(batch, seq, heads, stride, pad):
    _check_forward(batch, seq, heads, stride, pad)


def test_forward_random_shapes_and_strides():
    rng = np.random.default_rng(20241)
    for case in range(10):
        batch, heads = int(rng.integers(1, 3)), int(rng.integers(1, 3))
        seq = 128 * int(rng.integers(1, 7))
        stride = 64 * int(rng.integers(1, 9))
        _check_forward(batch, seq, heads, stride, 8 * int(rng.integers(0, 2)), seed=5000 + case)


def _check_forward(batch, seq, heads, stride, pad, seed=None):
    p = mst_inputs.attention_problem(batch, seq, heads, 64, seed=900 + seq + stride if seed is None else seed)
    out, lse = _run(p, stride, pad=pad)
    Q, K, V = p.split()
    ref, lse_ref = att.strided_attention(Q, K, V, stride)
    assert rel_err(out, ref) <= TOL["bf16"]
    np.testing.assert_allclose(lse, lse_ref, rtol=0, atol=2e-3)
    # no NaN anywhere and the first position copies its own value row
    assert np.isfinite(out).all()
    np.testing.assert_array_equal(out[:, :, 0], V[:, :, 0])


@pytest.mark.parametrize("kernel", ["warp", "tcgen05"])
def test_larger_scores_and_run_to_run_identity(kernel, monkeypatch):
    monkeypatch.setenv("MST_ATTN_FWD", kernel)
    p = mst_inputs.attention_problem(2, 512, 2, 64, seed=77, std=2.0)      # scaled scores of variance 16: peaked rows
    a, _ = _run(p, 256, want_lse=False)
    b, _ = _run(p, 256, want_lse=False)
    np.testing.assert_array_equal(a.view(np.uint32), b.view(np.uint32))
    Q, K, V = p.split()
    ref, _ = att.strided_attention(Q, K, V, 256)
    assert rel_err(a, ref) <= TOL["bf16"]


@pytest.mark.parametrize("kernel", ["warp", "tcgen05"])
@pytest.mark.parametrize("stride", [256, 128])
def test_gpt2_small_full_size_sampled(stride, kernel, monkeypatch):
    monkeypatch.setenv("MST_ATTN_FWD", kernel)
    # 16 sequences of 1024 tokens, 12 heads: the attention input of the benchmark's 16384-token batch
    rng = np.random.default_rng(12 + stride)
    p = mst_inputs.attention_problem(16, 1024, 12, 64)
    out, _ = _run(p, stride, want_lse=False)
    Q, K, V = p.split()
    n = 400
    b = rng.integers(0, 16, n); h = rng.integers(0, 12, n); i = rng.integers(0, 1024, n)
    i[:8] = [0, 127, 128, 255, 256, 511, 768, 1023]
    ref = att.strided_attention_at(Q, K, V, stride, b, h, i)
    assert rel_err(out[b, h, i], ref) <= TOL["bf16"]


def test_argument_errors():
    p = mst_inputs.attention_problem(1, 128, 1, 64)
    x = torch.zeros((128, 192), dtype=torch.bfloat16, device=dev())
    o = torch.zeros((128, 64), dtype=torch.bfloat16, device=dev())
    for kwargs in (dict(seq_len=100), dict(head_dim=32), dict(stride=96), dict(stride=0), dict(ld=60)):
        a = dict(ld=192, batch=1, seq_len=128, heads=1, head_dim=64, stride=128)
        a.update(kwargs)
        with pytest.raises(mst.MstError) as e:
            mst.mst_strided_attention_fwd(x, x.data_ptr() + 128, x.data_ptr() + 256, a["ld"], a["batch"], a["seq_len"],
                                          a["heads"], a["head_dim"], a["stride"], o, 64)
        assert e.value.status == 2          # MST_ERR_SHAPE
    mst.mst_strided_attention_fwd(x, x.data_ptr() + 128, x.data_ptr() + 256, 192, 0, 128, 1, 64, 128, o, 64)   # empty batch
