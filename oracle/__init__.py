"""CPU checker ("oracle") for the masked fully-connected layer path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA library never calls it and shares
no code with it.

The arithmetic lives in ``mst_oracle.cpp`` (plain C++, fp64, OpenMP); this
module compiles it with g++ on first use and exposes numpy-facing wrappers.
All inputs are the stored-precision values (fp32, or bf16 widened exactly)
converted to float64 before the sums are taken.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mst_oracle.cpp")
_LIB_PATH = os.path.join(_HERE, "_build", "libmst_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C++ checker into ``oracle/_build/libmst_oracle.so`` (g++ -O2 -fopenmp)."""
    os.makedirs(os.path.dirname(_LIB_PATH), exist_ok=True)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


_i64 = ctypes.c_int64
_u64 = ctypes.c_uint64
_dp = ctypes.POINTER(ctypes.c_double)
_fp = ctypes.POINTER(ctypes.c_float)
_bp = ctypes.POINTER(ctypes.c_uint8)
_ip = ctypes.POINTER(ctypes.c_int64)


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            L.mst_oracle_fwd.argtypes = [_i64, _i64, _i64, _dp, _dp, _bp, _dp]
            L.mst_oracle_bwd_x.argtypes = [_i64, _i64, _i64, _dp, _dp, _bp, _dp]
            L.mst_oracle_dw.argtypes = [_i64, _i64, _i64, _dp, _dp, _bp, _dp]
            L.mst_oracle_dense_grad.argtypes = [_i64, _i64, _i64, _dp, _dp, _dp]
            L.mst_oracle_fwd_at.argtypes = [_i64, _i64, _dp, _dp, _bp, _i64, _ip, _ip, _dp]
            L.mst_oracle_bwd_x_at.argtypes = [_i64, _i64, _dp, _dp, _bp, _i64, _ip, _ip, _dp]
            L.mst_oracle_grad_at.argtypes = [_i64, _i64, _i64, _dp, _dp, _i64, _ip, _ip, _dp]
            L.mst_oracle_stream.argtypes = [_u64, _u64, _i64]
            L.mst_oracle_stream.restype = _u64
            L.mst_oracle_rand_key.argtypes = [_u64, _i64]
            L.mst_oracle_rand_key.restype = _u64
            L.mst_oracle_mg_counts.argtypes = [ctypes.c_double, _i64, _i64, _i64, ctypes.c_double, _ip]
            L.mst_oracle_mg_counts.restype = ctypes.c_int
            L.mst_oracle_mg_update.argtypes = [_i64, _i64, _fp, _bp, _fp, _i64, _i64, _i64, _u64, _u64, _i64,
                                               ctypes.c_int, _ip, _ip, _ip, ctypes.c_float]
            L.mst_oracle_mg_update.restype = ctypes.c_int
            _lib = L
    return _lib


def _d(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _m(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint8)


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(t)


def threads() -> int:
    """Number of OpenMP threads the checker will use (the cores this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


# ------------------------------------------------------------------ products
def fwd(X, W, M) -> np.ndarray:
    """Y = X (W . M)^T in fp64.  X [T,I], W [O,I], M [O,I] -> Y [T,O]."""
    X, W, M = _d(X), _d(W), _m(M)
    T, I = X.shape
    O = W.shape[0]
    assert W.shape == (O, I) and M.shape == (O, I)
    Y = np.empty((T, O), dtype=np.float64)
    lib().mst_oracle_fwd(T, O, I, _p(X, _dp), _p(W, _dp), _p(M, _bp), _p(Y, _dp))
    return Y


def bwd_x(dY, W, M) -> np.ndarray:
    """dX = dY (W . M) in fp64.  dY [T,O] -> dX [T,I]."""
    dY, W, M = _d(dY), _d(W), _m(M)
    T, O = dY.shape
    I = W.shape[1]
    assert W.shape == (O, I) and M.shape == (O, I)
    dX = np.empty((T, I), dtype=np.float64)
    lib().mst_oracle_bwd_x(T, O, I, _p(dY, _dp), _p(W, _dp), _p(M, _bp), _p(dX, _dp))
    return dX


def dw(dY, X, M) -> np.ndarray:
    """dW = (dY^T X) . M in fp64, dense [O,I] with exact zeros off the mask."""
    dY, X, M = _d(dY), _d(X), _m(M)
    T, O = dY.shape
    I = X.shape[1]
    assert X.shape[0] == T and M.shape == (O, I)
    out = np.empty((O, I), dtype=np.float64)
    lib().mst_oracle_dw(T, O, I, _p(dY, _dp), _p(X, _dp), _p(M, _bp), _p(out, _dp))
    return out


def dense_grad(dY, X) -> np.ndarray:
    """G = dY^T X in fp64, dense [O,I]."""
    dY, X = _d(dY), _d(X)
    T, O = dY.shape
    I = X.shape[1]
    assert X.shape[0] == T
    G = np.empty((O, I), dtype=np.float64)
    lib().mst_oracle_dense_grad(T, O, I, _p(dY, _dp), _p(X, _dp), _p(G, _dp))
    return G


def _idx(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int64)


def fwd_at(X, W, M, t_idx, o_idx) -> np.ndarray:
    X, W, M, t_idx, o_idx = _d(X), _d(W), _m(M), _idx(t_idx), _idx(o_idx)
    O, I = W.shape
    out = np.empty(len(t_idx), dtype=np.float64)
    lib().mst_oracle_fwd_at(O, I, _p(X, _dp), _p(W, _dp), _p(M, _bp), len(t_idx), _p(t_idx, _ip), _p(o_idx, _ip),
                            _p(out, _dp))
    return out


def bwd_x_at(dY, W, M, t_idx, i_idx) -> np.ndarray:
    dY, W, M, t_idx, i_idx = _d(dY), _d(W), _m(M), _idx(t_idx), _idx(i_idx)
    O, I = W.shape
    out = np.empty(len(t_idx), dtype=np.float64)
    lib().mst_oracle_bwd_x_at(O, I, _p(dY, _dp), _p(W, _dp), _p(M, _bp), len(t_idx), _p(t_idx, _ip),
                              _p(i_idx, _ip), _p(out, _dp))
    return out


def grad_at(dY, X, o_idx, i_idx) -> np.ndarray:
    """sum_t dY[t,o] X[t,i] at the listed (o,i) pairs."""
    dY, X, o_idx, i_idx = _d(dY), _d(X), _idx(o_idx), _idx(i_idx)
    T, O = dY.shape
    I = X.shape[1]
    out = np.empty(len(o_idx), dtype=np.float64)
    lib().mst_oracle_grad_at(T, O, I, _p(dY, _dp), _p(X, _dp), len(o_idx), _p(o_idx, _ip), _p(i_idx, _ip),
                             _p(out, _dp))
    return out


# ------------------------------------------------------------ Mixed-Growing
def rand_key(seed: int, step: int, layer_id: int, flat_index: int) -> int:
    L = lib()
    return int(L.mst_oracle_rand_key(L.mst_oracle_stream(seed, step, layer_id), flat_index))


def mg_counts(zeta: float, nnz: int, n_target: int, numel: int, R: float) -> Tuple[int, int, int, int]:
    """(n_prune, n_grow, n_rand, n_grad) of Algorithm 1; raises ValueError when infeasible."""
    out = np.zeros(4, dtype=np.int64)
    rc = lib().mst_oracle_mg_counts(float(zeta), int(nnz), int(n_target), int(numel), float(R), _p(out, _ip))
    if rc != 0:
        raise ValueError("infeasible topology-update counts")
    return tuple(int(v) for v in out)


class NonFinite(ValueError):
    pass


def mg_update(W, M, G: Optional[np.ndarray], n_prune: int, n_grad: int, n_rand: int, seed: int, step: int,
              layer_id: int, allow_regrow_pruned: bool = False, prune_grad_weight: float = 0.0):
    """One Mixed-Growing update.  Returns (W_new f32 [O,I], M_new u8 [O,I], I_prune, I_grad, I_rand)."""
    W = np.array(W, dtype=np.float32, order="C", copy=True)
    M = np.array(M, dtype=np.uint8, order="C", copy=True)
    O, I = W.shape
    assert M.shape == (O, I)
    Gp = None
    if G is not None:
        G = np.ascontiguousarray(G, dtype=np.float32)
        assert G.shape == (O, I)
        Gp = _p(G, _fp)
    ip = np.zeros(max(n_prune, 1), dtype=np.int64)
    ig = np.zeros(max(n_grad, 1), dtype=np.int64)
    ir = np.zeros(max(n_rand, 1), dtype=np.int64)
    rc = lib().mst_oracle_mg_update(O, I, _p(W, _fp), _p(M, _bp), Gp, int(n_prune), int(n_grad), int(n_rand),
                                    int(seed), int(step), int(layer_id), int(bool(allow_regrow_pruned)),
                                    _p(ip, _ip), _p(ig, _ip), _p(ir, _ip), float(prune_grad_weight))
    if rc == 1:
        raise NonFinite("non-finite |w| or |g| in a selection key")
    if rc != 0:
        raise ValueError("infeasible topology update")
    return W, M, ip[:n_prune], ig[:n_grad], ir[:n_rand]


def to_csr(W, M):
    """Canonical CSR of W . M: rows ascending, columns ascending.  Returns (row_ptr i32, col_idx i32, vals)."""
    M = _m(M)
    W = np.ascontiguousarray(W)
    rows, cols = np.nonzero(M)          # row-major order
    row_ptr = np.zeros(M.shape[0] + 1, dtype=np.int32)
    np.cumsum(np.bincount(rows, minlength=M.shape[0]), out=row_ptr[1:])
    return row_ptr, cols.astype(np.int32), W[rows, cols]
