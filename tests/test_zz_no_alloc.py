"""The allocation-free mask -> CSR entry point against the regular pack + export path (needs a GPU).

Some users of the library may not allocate device memory at all (a framework that owns the whole GPU through its
own pool, a latency-critical loop, a thread running beside a stream capture).  ``mst_mask_to_csr_noalloc`` serves
them from a fixed work area inside the library.  Because that area is shared and keeps whatever the previous call
left in it, the check is made on two calls in a row with different layers: the second must not be disturbed by the
leftovers of the first.  The file name sorts last so that it runs after every other test.
"""
import numpy as np
import pytest

import mst_inputs

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    import paper_2408_11746_b200 as mst
    from gpu_util import dev, export_csr, make_layer, mdtype, tdtype, to_dev


_warmed = []


def _noalloc_csr(p, capacity):
    O, I = p.out_features, p.in_features
    rp = torch.full((O + 1,), -7, dtype=torch.int32, device=dev())
    ci = torch.full((max(capacity, 1),), -7, dtype=torch.int32, device=dev())
    vv = torch.zeros((max(capacity, 1),), dtype=tdtype(p), device=dev())
    W, M = to_dev(p, "W"), torch.from_numpy(p.mask).to(dev())
    if not _warmed:
        # the first call on a device looks up the work area's address; it is documented to come before any capture and
        # is not part of the no-allocation claim checked below
        mst.mst_mask_to_csr_noalloc(O, I, mdtype(p), W, I, M, capacity, rp, ci, vv)
        torch.cuda.synchronize()
        _warmed.append(True)
    # the call's contract: no device memory is allocated or freed, neither through torch's allocator nor around it
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    stats0 = torch.cuda.memory_stats()
    mst.mst_mask_to_csr_noalloc(O, I, mdtype(p), W, I, M, capacity, rp, ci, vv)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    stats1 = torch.cuda.memory_stats()
    assert free1 == free0
    for key in ("allocation.all.allocated", "allocation.all.freed", "segment.all.allocated", "segment.all.freed"):
        assert stats1.get(key, 0) == stats0.get(key, 0), key
    return rp, ci, vv


def _bits(v, p, n):
    v = v[:n]
    return v.view(torch.int16).cpu().numpy().view(np.uint16) if p.dtype == "bf16" else v.cpu().numpy().view(np.uint32)


def test_noalloc_matches_pack_export_on_two_calls_in_a_row():
    # a larger layer first, then a smaller one of another dtype: stale words of the first stay in the work area
    cases = [mst_inputs.uniform_layer("a", 0, 1024, 768, 4, "bf16", 0.25, 11),
             mst_inputs.zipf_layer("b", 1, 130, 257, 4, "f32", 0.1, 12)]
    for p in cases:
        L = make_layer(p)
        rp_ref, ci_ref, vb_ref = export_csr(L, p.dtype)
        L.close()
        rp, ci, vv = _noalloc_csr(p, p.nnz)
        np.testing.assert_array_equal(rp.cpu().numpy(), rp_ref)
        np.testing.assert_array_equal(ci[: p.nnz].cpu().numpy(), ci_ref)
        np.testing.assert_array_equal(_bits(vv, p, p.nnz), vb_ref)          # values are moved, not computed: bit-exact


def test_noalloc_capacity_and_size_limits():
    p = mst_inputs.uniform_layer("c", 0, 64, 96, 4, "f32", 0.5, 13)
    cap = p.nnz // 2
    rp, ci, vv = _noalloc_csr(p, cap)
    assert int(rp[-1]) == p.nnz                      # the true count is still reported
    L = make_layer(p)
    _, ci_ref, _ = export_csr(L, p.dtype)
    L.close()
    np.testing.assert_array_equal(ci[:cap].cpu().numpy(), ci_ref[:cap])
    # beyond the fixed work area: refused on the host, nothing launched
    d = torch.zeros(8, device=dev())
    with pytest.raises(mst.MstError) as e:
        mst.mst_mask_to_csr_noalloc(4097, 1024, mst.MST_F32, d, 1024, d, 8, d, d, d)
    assert e.value.status == 4
    with pytest.raises(mst.MstError) as e:
        mst.mst_mask_to_csr_noalloc(16, 16, mst.MST_F32, d, 8, d, 8, d, d, d)      # ldw < I
    assert e.value.status == 2
