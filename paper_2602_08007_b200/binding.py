"""ctypes binding of libtsr (see include/tsr.h).  Argument marshalling only: every step of the
optimizer path runs in the CUDA library.  PyTorch is used for device memory and streams.

The module-level functions carry the C names (tsr_create, tsr_project_core, ...) and take the
same arguments with ctypes structures; `Plan` is a small convenience holder that allocates the
state tensors with torch and passes their pointers.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libtsr.so")
_lib = None

TSR_OK = 0
TSR_F32, TSR_BF16 = 0, 1
TSR_RULE_ADAM, TSR_RULE_SGD = 0, 1
TSR_BLOCK_REEXPRESS_MOMENT = 1
TSR_BLOCK_ONE_SIDED = 2

STATUS_NAMES = {
    0: "TSR_OK", 1: "TSR_ERR_INVALID_ARG", 2: "TSR_ERR_SHAPE", 3: "TSR_ERR_ALIGNMENT", 4: "TSR_ERR_WORKSPACE",
    5: "TSR_ERR_CUDA", 6: "TSR_ERR_UNSUPPORTED", 7: "TSR_ERR_NOT_CONVERGED", 8: "TSR_ERR_RANK_DEFICIENT",
    9: "TSR_ERR_NONFINITE", 10: "TSR_ERR_TIMEOUT", 11: "TSR_ERR_NOT_BOUND",
}


class MatDesc(ctypes.Structure):
    _fields_ = [("m", ctypes.c_int64), ("n", ctypes.c_int64), ("ldg", ctypes.c_int64), ("ldw", ctypes.c_int64),
                ("r", ctypes.c_int32), ("p", ctypes.c_int32), ("q", ctypes.c_int32), ("K", ctypes.c_int32),
                ("g_dtype", ctypes.c_int32), ("w_dtype", ctypes.c_int32), ("is_embedding", ctypes.c_int32),
                ("flags", ctypes.c_int32)]


class MatPtrs(ctypes.Structure):
    _fields_ = [("G", ctypes.c_void_p), ("W", ctypes.c_void_p), ("U", ctypes.c_void_p), ("V", ctypes.c_void_p),
                ("M", ctypes.c_void_p), ("Vm", ctypes.c_void_p), ("C", ctypes.c_void_p)]


class DenseTensor(ctypes.Structure):
    _fields_ = [("param", ctypes.c_void_p), ("grad", ctypes.c_void_p), ("m", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("count", ctypes.c_int64), ("g_dtype", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class Hyper(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
                ("weight_decay", ctypes.c_float), ("scale", ctypes.c_float), ("step", ctypes.c_int64),
                ("rule", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class Limits(ctypes.Structure):
    _fields_ = [("wait_clocks", ctypes.c_int64), ("max_sweeps", ctypes.c_int32), ("sweep_block", ctypes.c_int32),
                ("starve_block", ctypes.c_int32), ("projection_launches", ctypes.c_int32)]


EXPORTS = [
    "tsr_version", "tsr_status_string", "tsr_last_error", "tsr_create", "tsr_destroy", "tsr_workspace_bytes",
    "tsr_bind", "tsr_bases_changed", "tsr_init_subspace", "tsr_project_core", "tsr_adam_core_step",
    "tsr_backproject_apply", "tsr_rsvd_refresh", "tsr_embed_step", "tsr_init_subspace_grouped",
    "tsr_project_core_grouped", "tsr_adam_core_step_grouped", "tsr_backproject_apply_grouped",
    "tsr_rsvd_refresh_grouped", "tsr_embed_step_grouped", "tsr_step_grouped", "tsr_step_grouped_host",
    "tsr_comm_bytes", "tsr_state_elems", "tsr_poll_status", "tsr_generate_omega", "tsr_block_uses_tensor_cores",
    "tsr_set_profiling", "tsr_get_stage_ms", "tsr_launch_count", "tsr_project_core_static", "tsr_dense_adamw",
    "tsr_set_limits", "tsr_refresh_gram",
]


class TsrError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, str(status)), message))
        self.status = status


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """Loads libtsr.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("libtsr.so is not built: run `python -m paper_2602_08007_b200.build` "
                              "(needs nvcc with sm_100a support)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64
        P = ctypes.POINTER
        L.tsr_version.restype = ctypes.c_int
        L.tsr_status_string.restype = ctypes.c_char_p
        L.tsr_status_string.argtypes = [ctypes.c_int]
        L.tsr_last_error.restype = ctypes.c_char_p
        L.tsr_last_error.argtypes = [vp]
        L.tsr_create.argtypes = [P(vp), P(MatDesc), i32]
        L.tsr_destroy.argtypes = [vp]
        L.tsr_workspace_bytes.argtypes = [vp, P(ctypes.c_size_t), P(ctypes.c_size_t)]
        L.tsr_bind.argtypes = [vp, P(MatPtrs), i32, vp, ctypes.c_size_t]
        L.tsr_bases_changed.argtypes = [vp, P(i32), i32, vp]
        L.tsr_init_subspace.argtypes = [vp, i32, u64, vp, vp]
        L.tsr_rsvd_refresh.argtypes = [vp, i32, u64, vp, vp]
        L.tsr_project_core.argtypes = [vp, i32, vp]
        L.tsr_adam_core_step.argtypes = [vp, i32, P(Hyper), vp]
        L.tsr_backproject_apply.argtypes = [vp, i32, P(Hyper), vp]
        L.tsr_embed_step.argtypes = [vp, i32, P(Hyper), u64, vp]
        L.tsr_init_subspace_grouped.argtypes = [vp, P(i32), i32, u64, P(vp), vp]
        L.tsr_rsvd_refresh_grouped.argtypes = [vp, P(i32), i32, u64, P(vp), vp]
        L.tsr_project_core_grouped.argtypes = [vp, P(i32), i32, vp]
        L.tsr_adam_core_step_grouped.argtypes = [vp, P(i32), i32, P(Hyper), vp]
        L.tsr_backproject_apply_grouped.argtypes = [vp, P(i32), i32, P(Hyper), vp]
        L.tsr_embed_step_grouped.argtypes = [vp, P(i32), i32, P(Hyper), u64, vp]
        L.tsr_step_grouped.argtypes = [vp, P(Hyper), u64, i32, vp]
        L.tsr_step_grouped_host.argtypes = [vp, P(vp), vp, P(Hyper), u64, i32, vp]
        L.tsr_comm_bytes.argtypes = [vp, i64, i32, P(u64), P(u64)]
        L.tsr_state_elems.argtypes = [vp, P(u64)]
        L.tsr_poll_status.argtypes = [vp, P(i32), i32, vp]
        L.tsr_generate_omega.argtypes = [vp, i32, u64, vp, vp]
        L.tsr_block_uses_tensor_cores.argtypes = [vp, i32]
        L.tsr_block_uses_tensor_cores.restype = i32
        L.tsr_set_profiling.argtypes = [vp, i32]
        L.tsr_get_stage_ms.argtypes = [vp, P(ctypes.c_float), i32]
        L.tsr_launch_count.argtypes = [vp, P(u64)]
        L.tsr_project_core_static.argtypes = [vp, i32, i64, i64, i64, vp, vp, i32, vp, vp]
        L.tsr_dense_adamw.argtypes = [P(DenseTensor), i32, P(Hyper), vp]
        L.tsr_set_limits.argtypes = [vp, P(Limits)]
        L.tsr_refresh_gram.argtypes = [vp, i32, i32, vp, vp, vp]
        _lib = L
    return _lib


def make_hyper(step: int, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
               weight_decay: float = 0.0, scale: float = 1.0, rule: int = TSR_RULE_ADAM) -> Hyper:
    return Hyper(lr, beta1, beta2, eps, weight_decay, scale, step, rule, 0)


def _field(b, name, default=None):
    if isinstance(b, dict):
        return b.get(name, default)
    return getattr(b, name, default)


def _idx_array(idx: Optional[Sequence[int]]):
    if idx is None:
        return None, 0
    arr = (ctypes.c_int32 * len(idx))(*idx)
    return arr, len(idx)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


STATIC_SCRATCH_FLOATS = 1 << 20


def project_core_static(G: torch.Tensor, U: torch.Tensor, V: torch.Tensor, C: torch.Tensor, stream=None) -> None:
    """C = U^T G V through tsr_project_core_static: no context, no workspace, no allocation --
    for callers that are not allowed to allocate device memory.  G is a 2-D (possibly row-padded)
    FP32 or BF16 tensor, U (m x r), V (n x r) and C (r x r) dense FP32, all on the current device."""
    if G.dim() != 2 or U.dim() != 2 or V.dim() != 2 or C.dim() != 2:
        raise ValueError("G, U, V and C must be matrices")
    m, n = G.shape
    r = U.shape[1]
    if G.dtype not in (torch.float32, torch.bfloat16) or G.stride(1) != 1 or G.stride(0) < n:
        raise ValueError("G must be FP32 or BF16 with unit column stride")
    if tuple(U.shape) != (m, r) or tuple(V.shape) != (n, r) or tuple(C.shape) != (r, r):
        raise ValueError("shapes must be U (m, r), V (n, r), C (r, r) for G (m, n)")
    for t in (U, V, C):
        if t.dtype != torch.float32 or not t.is_contiguous():
            raise ValueError("U, V and C must be contiguous FP32 tensors")
    if not all(t.is_cuda and t.device == G.device for t in (G, U, V, C)):
        raise ValueError("all tensors must live on the same CUDA device")
    dt = TSR_BF16 if G.dtype == torch.bfloat16 else TSR_F32
    rc = lib().tsr_project_core_static(ctypes.c_void_p(G.data_ptr()), dt, m, n, G.stride(0),
                                       ctypes.c_void_p(U.data_ptr()), ctypes.c_void_p(V.data_ptr()), r,
                                       ctypes.c_void_p(C.data_ptr()), _stream_ptr(stream))
    if rc != TSR_OK:
        raise TsrError(rc, "tsr_project_core_static")


def dense_adamw(params, grads, ms, vs, hyper: Hyper, stream=None) -> None:
    """tsr_dense_adamw over lists of torch tensors (params / ms / vs FP32, grads FP32 or BF16,
    all contiguous and on the current device), updated in place."""
    n = len(params)
    arr = (DenseTensor * max(n, 1))()
    for i in range(n):
        assert params[i].is_contiguous() and grads[i].is_contiguous() and params[i].dtype == torch.float32
        arr[i] = DenseTensor(params[i].data_ptr(), grads[i].data_ptr(), ms[i].data_ptr(), vs[i].data_ptr(),
                             params[i].numel(), TSR_BF16 if grads[i].dtype == torch.bfloat16 else TSR_F32, 0)
    rc = lib().tsr_dense_adamw(arr, n, ctypes.byref(hyper), _stream_ptr(stream))
    if rc != TSR_OK:
        raise TsrError(rc, "tsr_dense_adamw")


class Plan:
    """Owns a tsr_ctx plus the torch tensors it is bound to.

    blocks: sequence of dicts/objects with m, n, r, p, q, K (and optionally is_embedding, flags).
    g_dtype: torch.float32 or torch.bfloat16.  w_dtype: torch.float32 (master weights) or
    torch.bfloat16.  Leading dimensions are padded to 16-byte row pitches unless pad=False.
    """

    def __init__(self, blocks, g_dtype=torch.bfloat16, device="cuda", pad: bool = True, gradients=None,
                 weights=None, w_dtype=torch.float32):
        L = lib()
        self.device = torch.device(device)
        self.g_dtype = g_dtype
        self.w_dtype = w_dtype
        wes = 2 if w_dtype == torch.bfloat16 else 4
        self.blocks = list(blocks)
        nb = len(self.blocks)
        ges = 2 if g_dtype == torch.bfloat16 else 4
        self.descs = (MatDesc * nb)()
        self.G: List[torch.Tensor] = []
        self.W: List[torch.Tensor] = []
        self.U, self.V, self.M, self.Vm, self.C = [], [], [], [], []
        for i, b in enumerate(self.blocks):
            g = lambda name, default=None, _b=b: _field(_b, name, default)
            m, n, r = int(g("m")), int(g("n")), int(g("r"))
            if gradients is not None:
                G = gradients[i]
                ldg = G.stride(0)
            else:
                ldg = (n + (16 // ges) - 1) // (16 // ges) * (16 // ges) if pad else n
                G = torch.zeros(m, ldg, dtype=g_dtype, device=self.device)[:, :n]
            if weights is not None:
                Wt = weights[i]
                ldw = Wt.stride(0)
            else:
                ldw = (n + (16 // wes) - 1) // (16 // wes) * (16 // wes) if pad else n
                Wt = torch.zeros(m, ldw, dtype=w_dtype, device=self.device)[:, :n]
            self.G.append(G)
            self.W.append(Wt)
            self.U.append(torch.zeros(m, r, dtype=torch.float32, device=self.device))
            self.V.append(torch.zeros(n, r, dtype=torch.float32, device=self.device))
            cn = n if int(g("flags", 0)) & TSR_BLOCK_ONE_SIDED else r   # one-sided arm: the core is r x n
            self.M.append(torch.zeros(r, cn, dtype=torch.float32, device=self.device))
            self.Vm.append(torch.zeros(r, cn, dtype=torch.float32, device=self.device))
            self.C.append(torch.zeros(r, cn, dtype=torch.float32, device=self.device))
            self.descs[i] = MatDesc(m, n, ldg, ldw, r, int(g("p", 0)), int(g("q", 0)), int(g("K", 0)),
                                    TSR_BF16 if g_dtype == torch.bfloat16 else TSR_F32,
                                    TSR_BF16 if w_dtype == torch.bfloat16 else TSR_F32,
                                    1 if g("is_embedding", False) else 0, int(g("flags", 0)))
        self.ctx = ctypes.c_void_p()
        self._check(L.tsr_create(ctypes.byref(self.ctx), self.descs, nb), create=True)
        sb, rb = ctypes.c_size_t(), ctypes.c_size_t()
        self._check(L.tsr_workspace_bytes(self.ctx, ctypes.byref(sb), ctypes.byref(rb)))
        self.step_bytes, self.refresh_bytes = sb.value, rb.value
        self.workspace = torch.empty(sb.value + rb.value + 256, dtype=torch.uint8, device=self.device)
        self.bind()

    # -- plumbing ---------------------------------------------------------------------------
    def _check(self, status: int, create: bool = False):
        if status != TSR_OK:
            msg = "" if create or not self.ctx else lib().tsr_last_error(self.ctx).decode()
            raise TsrError(status, msg)

    def bind(self):
        nb = len(self.blocks)
        ptrs = (MatPtrs * nb)()
        for i in range(nb):
            vm = None if self.Vm[i] is None else self.Vm[i].data_ptr()   # None: a block that only ever runs TSR_RULE_SGD
            ptrs[i] = MatPtrs(self.G[i].data_ptr(), self.W[i].data_ptr(), self.U[i].data_ptr(), self.V[i].data_ptr(),
                              self.M[i].data_ptr(), vm, self.C[i].data_ptr())
        ws = self.workspace.data_ptr()
        ws_al = (ws + 255) // 256 * 256
        self._check(lib().tsr_bind(self.ctx, ptrs, nb, ctypes.c_void_p(ws_al), self.workspace.numel() - (ws_al - ws)))

    def close(self):
        if self.ctx:
            lib().tsr_destroy(self.ctx)
            self.ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C calls --------------------------------------------------------------------------
    def uses_tensor_cores(self, i: int) -> bool:
        return lib().tsr_block_uses_tensor_cores(self.ctx, i) == 1

    def bases_changed(self, idx=None, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_bases_changed(self.ctx, arr, cnt, _stream_ptr(stream)))

    def _omega_array(self, omegas):
        if omegas is None:
            return None
        arr = (ctypes.c_void_p * len(omegas))()
        for j, o in enumerate(omegas):
            arr[j] = None if o is None else o.data_ptr()
        return arr

    def init_subspace(self, idx=None, seed: int = 0, omegas=None, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_init_subspace_grouped(self.ctx, arr, cnt, seed, self._omega_array(omegas), _stream_ptr(stream)))

    def rsvd_refresh(self, idx=None, seed: int = 0, omegas=None, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_rsvd_refresh_grouped(self.ctx, arr, cnt, seed, self._omega_array(omegas), _stream_ptr(stream)))

    def project_core(self, idx=None, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_project_core_grouped(self.ctx, arr, cnt, _stream_ptr(stream)))

    def adam_core_step(self, hyper: Hyper, idx=None, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_adam_core_step_grouped(self.ctx, arr, cnt, ctypes.byref(hyper), _stream_ptr(stream)))

    def backproject_apply(self, hyper: Hyper, idx=None, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_backproject_apply_grouped(self.ctx, arr, cnt, ctypes.byref(hyper), _stream_ptr(stream)))

    def embed_step(self, hyper: Hyper, idx=None, seed: int = 0, stream=None):
        arr, cnt = _idx_array(idx)
        self._check(lib().tsr_embed_step_grouped(self.ctx, arr, cnt, ctypes.byref(hyper), seed, _stream_ptr(stream)))

    def step(self, hyper: Hyper, seed: int = 0, fuse_adam: bool = True, stream=None):
        self._check(lib().tsr_step_grouped(self.ctx, ctypes.byref(hyper), seed, 1 if fuse_adam else 0, _stream_ptr(stream)))

    def step_host(self, g_host: Sequence[torch.Tensor], c_host: Optional[torch.Tensor], hyper: Hyper, seed: int = 0,
                  fuse_adam: bool = True, stream=None):
        arr = (ctypes.c_void_p * len(g_host))(*[t.data_ptr() for t in g_host])
        cptr = None if c_host is None else ctypes.c_void_p(c_host.data_ptr())
        self._check(lib().tsr_step_grouped_host(self.ctx, arr, cptr, ctypes.byref(hyper), seed, 1 if fuse_adam else 0,
                                                _stream_ptr(stream)))

    def comm_bytes(self, step: int, bytes_per_elem: int = 4):
        core, sk = ctypes.c_uint64(), ctypes.c_uint64()
        self._check(lib().tsr_comm_bytes(self.ctx, step, bytes_per_elem, ctypes.byref(core), ctypes.byref(sk)))
        return core.value, sk.value

    def state_elems(self) -> int:
        e = ctypes.c_uint64()
        self._check(lib().tsr_state_elems(self.ctx, ctypes.byref(e)))
        return e.value

    def poll_status(self, stream=None) -> List[int]:
        nb = len(self.blocks)
        arr = (ctypes.c_int32 * nb)()
        self._check(lib().tsr_poll_status(self.ctx, arr, nb, _stream_ptr(stream)))
        return list(arr)

    def set_limits(self, wait_clocks: int = 0, max_sweeps: int = 0, sweep_block: int = -1, starve_block: int = -1,
                   projection_launches: int = 0):
        lim = Limits(wait_clocks, max_sweeps, sweep_block, starve_block, projection_launches)
        self._check(lib().tsr_set_limits(self.ctx, ctypes.byref(lim)))

    def refresh_gram(self, i: int, side: int, X: torch.Tensor, stream=None) -> torch.Tensor:
        """S = X^T X (FP64, k x k) through the Gram kernels the refresh of block i uses; X is FP32, rows x k with
        rows = m (side 0) or n (side 1).  Overwrites the block's refresh work buffers."""
        b = self.blocks[i]
        rows, k = int(_field(b, "n") if side else _field(b, "m")), int(_field(b, "r")) + int(_field(b, "p", 0))
        if X.dtype != torch.float32 or tuple(X.shape) != (rows, k) or not X.is_contiguous() or not X.is_cuda:
            raise ValueError("X must be a contiguous CUDA FP32 tensor of shape (%d, %d)" % (rows, k))
        S = torch.empty(k, k, dtype=torch.float64, device=X.device)
        self._check(lib().tsr_refresh_gram(self.ctx, i, side, X.data_ptr(), S.data_ptr(), _stream_ptr(stream)))
        return S

    def set_profiling(self, enable: bool):
        self._check(lib().tsr_set_profiling(self.ctx, 1 if enable else 0))

    def stage_ms(self) -> List[float]:
        arr = (ctypes.c_float * 6)()
        self._check(lib().tsr_get_stage_ms(self.ctx, arr, 6))
        return list(arr)

    def launch_count(self) -> int:
        c = ctypes.c_uint64()
        self._check(lib().tsr_launch_count(self.ctx, ctypes.byref(c)))
        return c.value

    def generate_omega(self, i: int, seed: int, stream=None) -> torch.Tensor:
        d = self.descs[i]
        out = torch.empty(d.n, d.r + d.p, dtype=torch.float32, device=self.device)
        self._check(lib().tsr_generate_omega(self.ctx, i, seed, ctypes.c_void_p(out.data_ptr()), _stream_ptr(stream)))
        return out
