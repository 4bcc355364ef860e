"""ctypes front end of the FP64 CPU oracle (tsr_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Every function takes and returns numpy float64 arrays (row-major).  Callers
widen BF16 / FP32 inputs exactly to FP64 first, so the oracle consumes the
same bits the CUDA library receives and does all arithmetic in FP64.

Nothing here imports the CUDA library or its binding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tsr_oracle.c")
_LIB = os.path.join(_HERE, "libtsr_oracle.so")
_lock = threading.Lock()
_lib = None

_i64 = ctypes.c_int64
_dbl = ctypes.c_double
_ptr = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile tsr_oracle.c with gcc (-O2, OpenMP) into libtsr_oracle.so beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"]
        subprocess.check_call(cmd)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.tsro_project_core.argtypes = [_i64, _i64, _i64, _ptr, _i64, _ptr, _ptr, _ptr]
            lib.tsro_project_one_sided.argtypes = [_i64, _i64, _i64, _ptr, _i64, _ptr, _ptr]
            lib.tsro_adam_core.argtypes = [_i64, _ptr, _ptr, _ptr, _ptr, _dbl, _dbl, _dbl, _i64]
            lib.tsro_sgd_core.argtypes = [_i64, _ptr, _ptr, _ptr, _dbl]
            lib.tsro_dense_adamw.argtypes = [_i64, _ptr, _ptr, _ptr, _ptr, _dbl, _dbl, _dbl, _dbl, _dbl, _i64]
            lib.tsro_backproject_apply.argtypes = [_i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr, _i64, _dbl, _dbl, _dbl]
            lib.tsro_backproject_one_sided.argtypes = [_i64, _i64, _i64, _ptr, _ptr, _ptr, _i64, _dbl, _dbl, _dbl]
            lib.tsro_orth.argtypes = [_i64, _i64, _ptr, _ptr, _ptr]
            lib.tsro_svd_jacobi.argtypes = [_i64, _i64, _ptr, _ptr, _ptr, _ptr, ctypes.c_int]
            lib.tsro_rsvd_refresh.argtypes = [_i64, _i64, _i64, _i64, _i64, _ptr, _i64, _ptr, _ptr, _ptr, _ptr]
            lib.tsro_reexpress_moment.argtypes = [_i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr, _ptr]
            lib.tsro_exact_svd_refresh.argtypes = [_i64, _i64, _i64, _ptr, _i64, _ptr, _ptr, _ptr]
            for name in ("tsro_core_bytes", "tsro_sketch_bytes", "tsro_state_elems"):
                getattr(lib, name).restype = ctypes.c_uint64
            lib.tsro_core_bytes.argtypes = [_i64, _i64]
            lib.tsro_sketch_bytes.argtypes = [_i64, _i64, _i64, _i64, _i64]
            lib.tsro_state_elems.argtypes = [_i64, _i64, _i64]
            lib.tsro_num_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def _f64(a, writeable: bool = False) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype != np.float64 or not a.flags.c_contiguous:
        if writeable:
            raise TypeError("in/out oracle arrays must be C-contiguous float64")
        a = np.ascontiguousarray(a, dtype=np.float64)
    return a


def _p(a: np.ndarray):
    return a.ctypes.data_as(_ptr)


def _check(rc: int, what: str) -> int:
    if rc < 0:
        raise RuntimeError("oracle %s failed with code %d" % (what, rc))
    return rc


def num_threads() -> int:
    return int(_load().tsro_num_threads())


def project_core(G, U, V) -> np.ndarray:
    """C = U^T G V (Algorithm 1, core projection)."""
    G, U, V = _f64(G), _f64(U), _f64(V)
    m, n = G.shape
    r = U.shape[1]
    assert U.shape == (m, r) and V.shape == (n, r)
    C = np.empty((r, r))
    _check(_load().tsro_project_core(m, n, r, _p(G), n, _p(U), _p(V), _p(C)), "project_core")
    return C


def project_one_sided(G, U) -> np.ndarray:
    """C = U^T G (the one-sided ablation arm)."""
    G, U = _f64(G), _f64(U)
    m, n = G.shape
    r = U.shape[1]
    C = np.empty((r, n))
    _check(_load().tsro_project_one_sided(m, n, r, _p(G), n, _p(U), _p(C)), "project_one_sided")
    return C


def adam_core(C, M, Vm, beta1, beta2, eps, t) -> np.ndarray:
    """Core-space Adam; M and Vm (float64, contiguous) are updated in place; returns D."""
    C = _f64(C)
    M, Vm = _f64(M, True), _f64(Vm, True)
    D = np.empty_like(C)
    _load().tsro_adam_core(C.size, _p(C), _p(M), _p(Vm), _p(D), beta1, beta2, eps, int(t))
    return D


def sgd_core(C, M, beta) -> np.ndarray:
    """Momentum core update of Algorithm 2; M updated in place; returns D = M."""
    C = _f64(C)
    M = _f64(M, True)
    D = np.empty_like(C)
    _load().tsro_sgd_core(C.size, _p(C), _p(M), _p(D), beta)
    return D


def dense_adamw(P, G, M, Vm, lr, beta1, beta2, eps, weight_decay, t) -> None:
    """Textbook AdamW on a dense parameter array; P, M, Vm (float64, contiguous) updated in place."""
    G = _f64(G)
    P, M, Vm = _f64(P, True), _f64(M, True), _f64(Vm, True)
    assert P.size == G.size == M.size == Vm.size
    _load().tsro_dense_adamw(P.size, _p(P), _p(G), _p(M), _p(Vm), lr, beta1, beta2, eps, weight_decay, int(t))


def backproject_apply(U, D, V, W, lr, weight_decay=0.0, scale=1.0) -> None:
    """W <- W - lr (scale * U D V^T + weight_decay * W), in place on the float64 array W."""
    U, D, V = _f64(U), _f64(D), _f64(V)
    W = _f64(W, True)
    m, n = W.shape
    r = U.shape[1]
    assert U.shape == (m, r) and V.shape == (n, r) and D.shape == (r, r)
    _check(_load().tsro_backproject_apply(m, n, r, _p(U), _p(D), _p(V), _p(W), n, lr, weight_decay, scale),
           "backproject_apply")


def backproject_one_sided(U, D, W, lr, weight_decay=0.0, scale=1.0) -> None:
    """One-sided arm (Table 1): W <- W - lr (scale * U D + weight_decay * W) with D of shape r x n,
    in place on the float64 array W."""
    U, D = _f64(U), _f64(D)
    W = _f64(W, True)
    m, n = W.shape
    r = U.shape[1]
    assert U.shape == (m, r) and D.shape == (r, n)
    _check(_load().tsro_backproject_one_sided(m, n, r, _p(U), _p(D), _p(W), n, lr, weight_decay, scale),
           "backproject_one_sided")


def orth(Y, return_r: bool = False):
    """Thin Householder QR: orthonormal Q (M x k) spanning the columns of Y."""
    Y = _f64(Y)
    M, k = Y.shape
    Q = np.empty((M, k))
    R = np.empty((k, k)) if return_r else None
    _check(_load().tsro_orth(M, k, _p(Y), _p(Q), _p(R) if return_r else None), "orth")
    return (Q, R) if return_r else Q


def svd_jacobi(B, max_sweeps: int = 60):
    """Thin SVD of a k x n matrix (k <= n): returns (Ut k x k, S k, Vt n x k), S descending."""
    B = _f64(B)
    k, n = B.shape
    Ut, S, Vt = np.empty((k, k)), np.empty(k), np.empty((n, k))
    _check(_load().tsro_svd_jacobi(k, n, _p(B), _p(Ut), _p(S), _p(Vt), max_sweeps), "svd_jacobi")
    return Ut, S, Vt


def rsvd_refresh(G, Omega, r, q):
    """Randomized-SVD refresh of the bases; Omega is n x (r+p).  Returns (U, V, sigma)."""
    G, Omega = _f64(G), _f64(Omega)
    m, n = G.shape
    k = Omega.shape[1]
    assert Omega.shape[0] == n and k >= r
    U, V, S = np.empty((m, r)), np.empty((n, r)), np.empty(k)
    _check(_load().tsro_rsvd_refresh(m, n, r, k - r, q, _p(G), n, _p(Omega), _p(U), _p(V), _p(S)),
           "rsvd_refresh")
    return U, V, S


def reexpress_moment(M, Uold, Vold, Unew, Vnew) -> None:
    """M <- Unew^T (Uold M Vold^T) Vnew, in place (optional moment re-expression at a refresh)."""
    M = _f64(M, True)
    Uold, Vold, Unew, Vnew = _f64(Uold), _f64(Vold), _f64(Unew), _f64(Vnew)
    m, r = Uold.shape
    n = Vold.shape[0]
    _check(_load().tsro_reexpress_moment(m, n, r, _p(Uold), _p(Vold), _p(Unew), _p(Vnew), _p(M)), "reexpress_moment")


def exact_svd_refresh(G, r):
    """Top-r singular vectors of G itself (the exact-SVD refresh arm)."""
    G = _f64(G)
    m, n = G.shape
    U, V, S = np.empty((m, r)), np.empty((n, r)), np.empty(min(m, n))
    _check(_load().tsro_exact_svd_refresh(m, n, r, _p(G), n, _p(U), _p(V), _p(S)), "exact_svd_refresh")
    return U, V, S


def core_bytes(r, bytes_per_elem=4) -> int:
    return int(_load().tsro_core_bytes(r, bytes_per_elem))


def sketch_bytes(m, n, r, p, bytes_per_elem=4) -> int:
    return int(_load().tsro_sketch_bytes(m, n, r, p, bytes_per_elem))


def state_elems(m, n, r) -> int:
    return int(_load().tsro_state_elems(m, n, r))


class OracleBlock:
    """State (U, V, m, v, W, t) of one matrix block, stepped as Algorithm 1 prescribes."""

    def __init__(self, W0, r, p, q, K, sgd: bool = False):
        self.W = np.array(W0, dtype=np.float64, order="C")
        self.m_rows, self.n_cols = self.W.shape
        self.r, self.p, self.q, self.K = int(r), int(p), int(q), int(K)
        self.M = np.zeros((r, r))
        self.Vm = np.zeros((r, r))
        self.U = None
        self.V = None
        self.t = 1
        self.sgd = sgd
        self.C = None
        self.D = None
        self.sigma = None

    def init_subspace(self, G0, Omega):
        self.U, self.V, self.sigma = rsvd_refresh(G0, Omega, self.r, self.q)

    def set_bases(self, U, V):
        self.U = np.array(U, dtype=np.float64, order="C")
        self.V = np.array(V, dtype=np.float64, order="C")

    def refresh_due(self) -> bool:
        return self.K > 0 and self.t % self.K == 0

    def refresh(self, G, Omega):
        self.U, self.V, self.sigma = rsvd_refresh(G, Omega, self.r, self.q)

    def step(self, G, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, scale=1.0, Omega=None,
             skip_refresh: bool = False):
        """One step on gradient G.  With skip_refresh the caller has already replaced the
        bases for this step (lock-step parity hands the GPU's refreshed bases over)."""
        if self.refresh_due() and not skip_refresh:
            if Omega is None:
                raise ValueError("refresh due at t=%d but no Omega given" % self.t)
            self.refresh(G, Omega)
        self.C = project_core(G, self.U, self.V)
        if self.sgd:
            self.D = sgd_core(self.C, self.M, beta1)
            backproject_apply(self.U, self.D, self.V, self.W, lr, 0.0, 1.0)
        else:
            self.D = adam_core(self.C, self.M, self.Vm, beta1, beta2, eps, self.t)
            backproject_apply(self.U, self.D, self.V, self.W, lr, weight_decay, scale)
        self.t += 1
