"""Helpers shared by the GPU parity tests: upload a LayerProblem, run the library, fetch results as numpy."""
import numpy as np
import torch

import paper_2408_11746_b200 as mst

TOL = {"f32": 1e-5, "bf16": 2e-2}     # max |gpu - ref| / max |ref|


def rel_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(got - ref)) / max(float(np.max(np.abs(ref))), 1e-300)) if ref.size else 0.0


def dev():
    return torch.device("cuda:0")


def to_dev(p, name, ld=None):
    """Upload X / W / dY of a LayerProblem in its stored dtype; optional padded leading dimension."""
    if p.dtype == "bf16":
        a = getattr(p, name + "_bits").view(np.int16)
        tdt = torch.bfloat16
    else:
        a = getattr(p, name)
        tdt = torch.float32
    t = torch.from_numpy(np.ascontiguousarray(a)).to(dev())
    if p.dtype == "bf16":
        t = t.view(tdt)
    if ld is not None and ld != t.shape[1]:
        buf = torch.full((t.shape[0], ld), float("nan"), dtype=tdt, device=dev())
        buf[:, : t.shape[1]] = t
        return buf
    return t


def tdtype(p):
    return torch.bfloat16 if p.dtype == "bf16" else torch.float32


def mdtype(p):
    return mst.MST_BF16 if p.dtype == "bf16" else mst.MST_F32


def make_layer(p, capacity=None):
    L = mst.Layer(p.layer_id, p.out_features, p.in_features, mdtype(p), capacity)
    Wd = to_dev(p, "W")
    Md = torch.from_numpy(p.mask).to(dev())
    L.pack(Wd, Md)
    return L


def host(t):
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def export_csr(L, p_dtype):
    nnz = L.nnz
    rp = torch.empty(L.out_features + 1, dtype=torch.int32, device=dev())
    ci = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev())
    vv = torch.empty(max(nnz, 1), dtype=torch.bfloat16 if p_dtype == "bf16" else torch.float32, device=dev())
    mst.mst_export_csr(L.handle, rp, ci, vv)
    torch.cuda.synchronize()
    v = vv[:nnz]
    vbits = v.view(torch.int16).cpu().numpy().view(np.uint16) if p_dtype == "bf16" else v.cpu().numpy().view(np.uint32)
    return rp.cpu().numpy(), ci[:nnz].cpu().numpy(), vbits


def export_csc(L):
    nnz = L.nnz
    cp = torch.empty(L.in_features + 1, dtype=torch.int32, device=dev())
    ri = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev())
    pm = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev())
    mst.mst_export_csc(L.handle, cp, ri, pm)
    torch.cuda.synchronize()
    return cp.cpu().numpy(), ri[:nnz].cpu().numpy(), pm[:nnz].cpu().numpy()


def value_bits(vals_f32, dtype):
    """Stored-precision bit patterns of reference values (already exactly representable)."""
    v = np.ascontiguousarray(vals_f32, dtype=np.float32)
    if dtype == "bf16":
        return (v.view(np.uint32) >> 16).astype(np.uint16)
    return v.view(np.uint32)
