"""Python binding of libmst (argument marshalling only; every step runs in the CUDA library).

The functions carry the names of the C entry points declared in ``include/mst.h``
and take device pointers as ``torch.Tensor`` (``data_ptr()`` is used) or plain
integers.  PyTorch appears only as the owner of device buffers and streams.

Importing the package needs ``libmst.so`` (built in-tree by
``python paper_2408_11746_b200/csrc/build.py``); there is no fallback path:
a missing library is an ImportError.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmst.so")

MST_F32, MST_BF16 = 0, 1
MST_PATH_AUTO, MST_PATH_CUDA_CORE, MST_PATH_TENSOR_CORE, MST_PATH_SPARSE_TC = 0, 1, 2, 3
MST_OK = 0
STATUS_NAMES = {0: "MST_OK", 1: "MST_ERR_INVALID_ARG", 2: "MST_ERR_SHAPE", 3: "MST_ERR_DTYPE", 4: "MST_ERR_CAPACITY",
                5: "MST_ERR_INFEASIBLE", 6: "MST_ERR_NONFINITE", 7: "MST_ERR_CORRUPT", 8: "MST_ERR_CUDA",
                9: "MST_ERR_NOT_PACKED"}
EXPORTS = ["mst_layer_create", "mst_layer_destroy", "mst_set_compute_path", "mst_layer_path_in_use", "mst_launch_count", "mst_track_values", "mst_values_changed", "mst_layer_nnz", "mst_pack", "mst_export_csr", "mst_export_csc",
           "mst_values", "mst_validate", "mst_spmm_fwd", "mst_spmm_bwd_x", "mst_spmm_fwd_gelu", "mst_spmm_bwd_x_gelu", "mst_strided_attention_fwd", "mst_strided_attention_bwd", "mst_sddmm_dw", "mst_dense_grad", "mst_sddmm_from_dense", "mst_dense_grad_dw",
           "mst_update_counts", "mst_rand_bracket", "mst_topology_update", "mst_topology_update_many", "mst_layer_step_host", "mst_layer_step_host_async", "mst_layer_step_host_wait", "mst_mask_to_csr_noalloc",
           "mst_device_error_flags", "mst_sv_sparsity", "mst_sv_update_fraction", "mst_er_densities",
           "mst_status_string"]


class MstError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%s)" % (where, STATUS_NAMES.get(status, status), status_string(status)))


class RegrowRule(ctypes.Structure):
    _fields_ = [("target_nnz", ctypes.c_int64), ("random_ratio", ctypes.c_double), ("seed", ctypes.c_uint64),
                ("step", ctypes.c_uint64), ("allow_regrow_pruned", ctypes.c_int32),
                ("prune_grad_weight", ctypes.c_float)]


class SvSchedule(ctypes.Structure):
    """S_M, N, Delta_W, T_U, Delta_R of the Sparsity-Variation schedule (paper defaults)."""
    _fields_ = [("max_sparsity", ctypes.c_double), ("n_stages", ctypes.c_int32), ("delta_w", ctypes.c_int64),
                ("t_ultra", ctypes.c_int64), ("delta_r", ctypes.c_int64)]

    def __init__(self, max_sparsity=0.96, n_stages=5, delta_w=2000, t_ultra=100000, delta_r=2000):
        super().__init__(max_sparsity, n_stages, delta_w, t_ultra, delta_r)


class UpdateStats(ctypes.Structure):
    _fields_ = [("nnz_before", ctypes.c_int64), ("nnz_after", ctypes.c_int64), ("n_prune", ctypes.c_int64),
                ("n_grad", ctypes.c_int64), ("n_rand", ctypes.c_int64), ("max_row_nnz", ctypes.c_int64)]


if not os.path.exists(LIB_PATH):
    raise ImportError("libmst.so is not built: run `python paper_2408_11746_b200/csrc/build.py` (needs nvcc); "
                      "there is no CPU fallback")
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i32, _i64, _f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
_sig = {
    "mst_layer_create": [ctypes.POINTER(_vp), _i32, _i32, _i32, ctypes.c_int, _i64],
    "mst_layer_destroy": [_vp],
    "mst_layer_nnz": [_vp, ctypes.POINTER(_i64)],
    "mst_set_compute_path": [_vp, ctypes.c_int],
    "mst_layer_path_in_use": [_vp, ctypes.POINTER(ctypes.c_int)],
    "mst_launch_count": [ctypes.POINTER(_i64)],
    "mst_track_values": [_vp, _i32],
    "mst_values_changed": [_vp],
    "mst_pack": [_vp, _vp, _i64, _vp, _vp],
    "mst_export_csr": [_vp, _vp, _vp, _vp, _vp],
    "mst_export_csc": [_vp, _vp, _vp, _vp, _vp],
    "mst_values": [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_i64)],
    "mst_validate": [_vp, _vp],
    "mst_spmm_fwd": [_vp, _vp, _i64, _i64, _vp, _i64, _vp],
    "mst_spmm_bwd_x": [_vp, _vp, _i64, _i64, _vp, _i64, _vp],
    "mst_spmm_fwd_gelu": [_vp, _vp, _i64, _i64, _vp, _i64, _vp, _i64, _vp],
    "mst_spmm_bwd_x_gelu": [_vp, _vp, _i64, _i64, _vp, _i64, _vp, _i64, _vp],
    "mst_strided_attention_fwd": [_vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32, _i32, _vp, _i64, _vp, _vp],
    "mst_strided_attention_bwd": [_vp, _vp, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp,
                                  _i64, _vp],
    "mst_sddmm_dw": [_vp, _vp, _i64, _vp, _i64, _i64, _vp, _vp],
    "mst_dense_grad": [_vp, _i64, _vp, _i64, _i64, _i32, _i32, ctypes.c_int, _vp, _vp],
    "mst_sddmm_from_dense": [_vp, _vp, _vp, _vp],
    "mst_dense_grad_dw": [_vp, _vp, _i64, _vp, _i64, _i64, _vp, _vp, _vp],
    "mst_update_counts": [_f64, _i64, _i64, _i64, _f64, ctypes.POINTER(_i64)],
    "mst_rand_bracket": [_i64, _i64, _f64, _i64, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(_i32)],
    "mst_topology_update": [_vp, _f64, ctypes.POINTER(RegrowRule), _vp, ctypes.POINTER(UpdateStats), _vp],
    "mst_topology_update_many": [_i32, ctypes.POINTER(_vp), ctypes.POINTER(_f64), ctypes.POINTER(RegrowRule), ctypes.POINTER(_vp),
                                 ctypes.POINTER(UpdateStats), _vp],
    "mst_layer_step_host": [_vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp],
    "mst_layer_step_host_async": [_vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp],
    "mst_layer_step_host_wait": [_vp],
    "mst_device_error_flags": [ctypes.POINTER(_i32)],
    "mst_sv_sparsity": [ctypes.POINTER(SvSchedule), _i64, ctypes.POINTER(_f64)],
    "mst_sv_update_fraction": [ctypes.POINTER(SvSchedule), _i64, _f64, _f64, ctypes.POINTER(_f64)],
    "mst_er_densities": [_i32, ctypes.POINTER(_i32), ctypes.POINTER(_i32), _f64, ctypes.POINTER(_f64)],
    "mst_mask_to_csr_noalloc": [_i32, _i32, ctypes.c_int, _vp, _i64, _vp, _i64, _vp, _vp, _vp, _vp],
}
for _n, _a in _sig.items():
    getattr(_lib, _n).argtypes = _a
    getattr(_lib, _n).restype = ctypes.c_int
_lib.mst_status_string.argtypes = [ctypes.c_int]
_lib.mst_status_string.restype = ctypes.c_char_p


def status_string(status: int) -> str:
    return _lib.mst_status_string(int(status)).decode()


def _ptr(x) -> Optional[int]:
    """Device (or host) address of a tensor / ndarray / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError("expected a tensor, an ndarray, an int address or None")


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(status: int, where: str) -> None:
    if status != MST_OK:
        raise MstError(status, where)


# ---------------------------------------------------------------- C entry points, same names
def mst_layer_create(layer_id: int, out_features: int, in_features: int, dtype: int, nnz_capacity: int) -> int:
    h = _vp()
    _check(_lib.mst_layer_create(ctypes.byref(h), layer_id, out_features, in_features, dtype, nnz_capacity),
           "mst_layer_create")
    return h.value


def mst_layer_destroy(layer: int) -> None:
    _check(_lib.mst_layer_destroy(layer), "mst_layer_destroy")


def mst_set_compute_path(layer: int, path: int) -> None:
    _check(_lib.mst_set_compute_path(layer, path), "mst_set_compute_path")


PATH_NAMES = {MST_PATH_AUTO: "auto", MST_PATH_CUDA_CORE: "cuda_core", MST_PATH_TENSOR_CORE: "dense_tiles",
              MST_PATH_SPARSE_TC: "sparse_tc"}


def path_name(path: int) -> str:
    return PATH_NAMES.get(path, "path %d" % path)


def mst_layer_path_in_use(layer: int) -> int:
    p = ctypes.c_int(0)
    _check(_lib.mst_layer_path_in_use(layer, ctypes.byref(p)), "mst_layer_path_in_use")
    return p.value


def mst_track_values(layer: int, enable: bool) -> None:
    _check(_lib.mst_track_values(layer, 1 if enable else 0), "mst_track_values")


def mst_values_changed(layer: int) -> None:
    _check(_lib.mst_values_changed(layer), "mst_values_changed")


def mst_launch_count() -> int:
    n = _i64(0)
    _check(_lib.mst_launch_count(ctypes.byref(n)), "mst_launch_count")
    return n.value


def mst_layer_nnz(layer: int) -> int:
    n = _i64()
    _check(_lib.mst_layer_nnz(layer, ctypes.byref(n)), "mst_layer_nnz")
    return n.value


def mst_pack(layer: int, W_dense, ldw: int, mask, stream=None) -> None:
    _check(_lib.mst_pack(layer, _ptr(W_dense), ldw, _ptr(mask), _stream(stream)), "mst_pack")


def mst_export_csr(layer: int, row_ptr, col_idx, vals, stream=None) -> None:
    _check(_lib.mst_export_csr(layer, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _stream(stream)), "mst_export_csr")


def mst_export_csc(layer: int, col_ptr, row_idx, perm, stream=None) -> None:
    _check(_lib.mst_export_csc(layer, _ptr(col_ptr), _ptr(row_idx), _ptr(perm), _stream(stream)), "mst_export_csc")


def mst_values(layer: int) -> Tuple[int, int]:
    p, n = _vp(), _i64()
    _check(_lib.mst_values(layer, ctypes.byref(p), ctypes.byref(n)), "mst_values")
    return p.value, n.value


def mst_validate(layer: int, stream=None) -> None:
    _check(_lib.mst_validate(layer, _stream(stream)), "mst_validate")


def mst_spmm_fwd(layer: int, X, ldx: int, T: int, Y, ldy: int, stream=None) -> None:
    _check(_lib.mst_spmm_fwd(layer, _ptr(X), ldx, T, _ptr(Y), ldy, _stream(stream)), "mst_spmm_fwd")


def mst_spmm_bwd_x(layer: int, dY, lddy: int, T: int, dX, lddx: int, stream=None) -> None:
    _check(_lib.mst_spmm_bwd_x(layer, _ptr(dY), lddy, T, _ptr(dX), lddx, _stream(stream)), "mst_spmm_bwd_x")


def mst_spmm_fwd_gelu(layer: int, X, ldx: int, T: int, Y_pre, ldpre: int, H, ldh: int, stream=None) -> None:
    _check(_lib.mst_spmm_fwd_gelu(layer, _ptr(X), ldx, T, _ptr(Y_pre), ldpre, _ptr(H), ldh,
                                  _stream(stream)), "mst_spmm_fwd_gelu")


def mst_spmm_bwd_x_gelu(layer: int, dY, lddy: int, T: int, Y_pre, ldpre: int, dPre, lddpre: int, stream=None) -> None:
    _check(_lib.mst_spmm_bwd_x_gelu(layer, _ptr(dY), lddy, T, _ptr(Y_pre), ldpre, _ptr(dPre), lddpre, _stream(stream)),
           "mst_spmm_bwd_x_gelu")


def mst_strided_attention_fwd(Q, K, V, ld: int, batch: int, seq_len: int, heads: int, head_dim: int, stride: int, Out,
                              ldo: int, lse=None, stream=None) -> None:
    _check(_lib.mst_strided_attention_fwd(_ptr(Q), _ptr(K), _ptr(V), ld, batch, seq_len, heads, head_dim, stride,
                                          _ptr(Out), ldo, _ptr(lse), _stream(stream)), "mst_strided_attention_fwd")


def mst_strided_attention_bwd(Q, K, V, ld: int, Out, ldo: int, dOut, lddo: int, lse, batch: int, seq_len: int, heads: int,
                              head_dim: int, stride: int, dQ, dK, dV, ldg: int, stream=None) -> None:
    _check(_lib.mst_strided_attention_bwd(_ptr(Q), _ptr(K), _ptr(V), ld, _ptr(Out), ldo, _ptr(dOut), lddo, _ptr(lse), batch,
                                          seq_len, heads, head_dim, stride, _ptr(dQ), _ptr(dK), _ptr(dV), ldg,
                                          _stream(stream)), "mst_strided_attention_bwd")


def mst_sddmm_dw(layer: int, dY, lddy: int, X, ldx: int, T: int, dW_vals, stream=None) -> None:
    _check(_lib.mst_sddmm_dw(layer, _ptr(dY), lddy, _ptr(X), ldx, T, _ptr(dW_vals), _stream(stream)), "mst_sddmm_dw")


def mst_dense_grad(dY, lddy: int, X, ldx: int, T: int, out_features: int, in_features: int, dtype: int, G,
                   stream=None) -> None:
    _check(_lib.mst_dense_grad(_ptr(dY), lddy, _ptr(X), ldx, T, out_features, in_features, dtype, _ptr(G),
                               _stream(stream)), "mst_dense_grad")


def mst_sddmm_from_dense(layer: int, G_dense, dW_vals, stream=None) -> None:
    _check(_lib.mst_sddmm_from_dense(layer, _ptr(G_dense), _ptr(dW_vals), _stream(stream)), "mst_sddmm_from_dense")


def mst_dense_grad_dw(layer: int, dY, lddy: int, X, ldx: int, T: int, G_dense, dW_vals, stream=None) -> None:
    _check(_lib.mst_dense_grad_dw(layer, _ptr(dY), lddy, _ptr(X), ldx, T, _ptr(G_dense), _ptr(dW_vals),
                                  _stream(stream)), "mst_dense_grad_dw")


def mst_update_counts(prune_frac: float, nnz: int, target_nnz: int, numel: int, random_ratio: float):
    """(n_prune, n_grow, n_rand, n_grad)."""
    out = (_i64 * 4)()
    _check(_lib.mst_update_counts(prune_frac, nnz, target_nnz, numel, random_ratio, out), "mst_update_counts")
    return tuple(int(v) for v in out)


def mst_rand_bracket(k: int, candidates: int, sigmas: float = 6.0, list_capacity: int = 32768):
    """(lo, hi) of the hash-key bracket planned for the k-th smallest of `candidates` uniform keys, or None."""
    lo, hi, planned = ctypes.c_uint64(), ctypes.c_uint64(), _i32()
    _check(_lib.mst_rand_bracket(k, candidates, sigmas, list_capacity, ctypes.byref(lo), ctypes.byref(hi), ctypes.byref(planned)),
           "mst_rand_bracket")
    return (int(lo.value), int(hi.value)) if planned.value else None


def mst_topology_update(layer: int, prune_frac: float, target_nnz: int = -1, random_ratio: float = 0.25,
                        seed: int = 0, step: int = 0, allow_regrow_pruned: bool = False, G_dense=None,
                        prune_grad_weight: float = 0.0,
                        want_stats: bool = True, stream=None) -> Optional[UpdateStats]:
    rule = RegrowRule(int(target_nnz), float(random_ratio), int(seed), int(step), int(bool(allow_regrow_pruned)),
                      float(prune_grad_weight))
    stats = UpdateStats() if want_stats else None
    _check(_lib.mst_topology_update(layer, float(prune_frac), ctypes.byref(rule), _ptr(G_dense),
                                    ctypes.byref(stats) if want_stats else None, _stream(stream)),
           "mst_topology_update")
    return stats


def mst_topology_update_many(layers, prune_frac, rules, G_dense, want_stats: bool = True, stream=None):
    """layers: handles; prune_frac: floats; rules: RegrowRule objects; G_dense: device arrays or None, one per layer."""
    n = len(layers)
    hs = (_vp * n)(*[int(h) for h in layers])
    zs = (_f64 * n)(*[float(z) for z in prune_frac])
    rs = (RegrowRule * n)(*rules)
    gs = (_vp * n)(*[_ptr(g) for g in G_dense])
    stats = (UpdateStats * n)() if want_stats else None
    _check(_lib.mst_topology_update_many(n, hs, zs, rs, gs, stats, _stream(stream)), "mst_topology_update_many")
    return list(stats) if want_stats else None


def mst_layer_step_host(layer: int, X_host, dY_host, T: int, Y_host, dX_host, dW_vals_host, stream=None) -> None:
    _check(_lib.mst_layer_step_host(layer, _ptr(X_host), _ptr(dY_host), T, _ptr(Y_host), _ptr(dX_host),
                                    _ptr(dW_vals_host), _stream(stream)), "mst_layer_step_host")


def mst_sv_sparsity(schedule: SvSchedule, step: int) -> float:
    out = _f64()
    _check(_lib.mst_sv_sparsity(ctypes.byref(schedule), step, ctypes.byref(out)), "mst_sv_sparsity")
    return out.value


def mst_sv_update_fraction(schedule: SvSchedule, step: int, zeta1: float = 0.3, decay: float = 1.0) -> float:
    out = _f64()
    _check(_lib.mst_sv_update_fraction(ctypes.byref(schedule), step, zeta1, decay, ctypes.byref(out)),
           "mst_sv_update_fraction")
    return out.value


def mst_er_densities(shapes, global_density: float):
    """shapes: [(out_features, in_features), ...] -> per-layer densities."""
    n = len(shapes)
    O = (_i32 * n)(*[int(o) for o, _ in shapes])
    I = (_i32 * n)(*[int(i) for _, i in shapes])
    d = (_f64 * n)()
    _check(_lib.mst_er_densities(n, O, I, global_density, d), "mst_er_densities")
    return [float(x) for x in d]


def mst_layer_step_host_async(layer: int, X_host, dY_host, T: int, Y_host, dX_host, dW_vals_host, stream=None) -> None:
    _check(_lib.mst_layer_step_host_async(layer, _ptr(X_host), _ptr(dY_host), T, _ptr(Y_host), _ptr(dX_host),
                                          _ptr(dW_vals_host), _stream(stream)), "mst_layer_step_host_async")


def mst_layer_step_host_wait(layer: int) -> None:
    _check(_lib.mst_layer_step_host_wait(layer), "mst_layer_step_host_wait")


def mst_device_error_flags() -> int:
    f = _i32()
    _check(_lib.mst_device_error_flags(ctypes.byref(f)), "mst_device_error_flags")
    return f.value


def mst_mask_to_csr_noalloc(out_features: int, in_features: int, dtype: int, W_dense, ldw: int, mask,
                            nnz_capacity: int, row_ptr, col_idx, vals, stream=None) -> None:
    """Dense mask -> CSR into caller-owned buffers, for callers that may not allocate device memory.

    The library works in a fixed internal array instead of allocating, so the layer is limited to
    4 194 304 entries, overlapping calls race, and the first call per device should happen outside
    stream capture.  See ``include/mst.h``.
    """
    _check(_lib.mst_mask_to_csr_noalloc(out_features, in_features, dtype, _ptr(W_dense), ldw, _ptr(mask),
                                        nnz_capacity, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _stream(stream)),
           "mst_mask_to_csr_noalloc")


# ---------------------------------------------------------------- small RAII convenience
class Layer:
    """Owns one ``mst_layer_t`` handle; methods forward to the entry points above."""

    def __init__(self, layer_id: int, out_features: int, in_features: int, dtype: int, nnz_capacity: Optional[int] = None):
        self.out_features, self.in_features, self.dtype = out_features, in_features, dtype
        cap = out_features * in_features if nnz_capacity is None else nnz_capacity
        self.handle = mst_layer_create(layer_id, out_features, in_features, dtype, cap)

    def close(self) -> None:
        if getattr(self, "handle", None):
            mst_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_path(self, path: int) -> None:
        mst_set_compute_path(self.handle, path)

    def track_values(self, enable: bool = True) -> None:
        mst_track_values(self.handle, enable)

    def values_changed(self) -> None:
        mst_values_changed(self.handle)

    def path_in_use(self) -> int:
        return mst_layer_path_in_use(self.handle)

    @property
    def nnz(self) -> int:
        return mst_layer_nnz(self.handle)

    def pack(self, W_dense, mask, ldw: Optional[int] = None, stream=None) -> None:
        mst_pack(self.handle, W_dense, self.in_features if ldw is None else ldw, mask, stream)

    def fwd(self, X, Y, T: int, stream=None) -> None:
        mst_spmm_fwd(self.handle, X, self.in_features, T, Y, self.out_features, stream)

    def bwd_x(self, dY, dX, T: int, stream=None) -> None:
        mst_spmm_bwd_x(self.handle, dY, self.out_features, T, dX, self.in_features, stream)

    def fwd_gelu(self, X, H, T: int, Y_pre=None, stream=None) -> None:
        mst_spmm_fwd_gelu(self.handle, X, self.in_features, T, Y_pre, self.out_features, H, self.out_features, stream)

    def bwd_x_gelu(self, dY, Y_pre, dPre, T: int, stream=None) -> None:
        mst_spmm_bwd_x_gelu(self.handle, dY, self.out_features, T, Y_pre, self.in_features, dPre, self.in_features, stream)

    def sddmm(self, dY, X, T: int, dW_vals, stream=None) -> None:
        mst_sddmm_dw(self.handle, dY, self.out_features, X, self.in_features, T, dW_vals, stream)

    def dense_grad(self, dY, X, T: int, G, stream=None) -> None:
        mst_dense_grad(dY, self.out_features, X, self.in_features, T, self.out_features, self.in_features, self.dtype,
                       G, stream)

    def dense_grad_dw(self, dY, X, T: int, G, dW_vals, stream=None) -> None:
        mst_dense_grad_dw(self.handle, dY, self.out_features, X, self.in_features, T, G, dW_vals, stream)

    def update(self, prune_frac: float, **kw):
        return mst_topology_update(self.handle, prune_frac, **kw)

    def validate(self, stream=None) -> None:
        mst_validate(self.handle, stream)
