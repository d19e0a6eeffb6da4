"""ctypes binding of libmwu.so: argument marshalling only.

Every function has the name and argument order of the C entry point in include/mwu.h and
passes raw device pointers of torch tensors.  There is no fallback: if the shared library is
missing or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmwu.so")

EXPORTS = ["mwu_status_string", "mwu_kernel_launches", "mwu_count_from_permille",
           "mwu_project_workspace_bytes", "mwu_project", "mwu_admm_step", "mwu_project_static",
           "mwu_packed_bytes", "mwu_pack", "mwu_gemm", "mwu_decode", "mwu_gemm_workspace_bytes",
           "mwu_gemm_ws", "mwu_conv_implicit", "mwu_conv_workspace_bytes", "mwu_conv_implicit_ws",
           "mwu_debug_conv_wait", "mwu_keep_n_of_m", "mwu_gemm_dense", "mwu_conv_dense_workspace_bytes",
           "mwu_conv_dense"]
MWU_STATIC_MAX_BLOCKS = 1048576

MWU_OK = 0
(MWU_ERR_INVALID_ARG, MWU_ERR_SHAPE, MWU_ERR_ALIGNMENT, MWU_ERR_WORKSPACE, MWU_ERR_UNSUPPORTED_DEVICE,
 MWU_ERR_CUDA) = 1, 2, 3, 4, 5, 6
MWU_DEV_NONFINITE, MWU_DEV_TIMEOUT, MWU_DEV_BOUNDS, MWU_DEV_SELECT = 1, 2, 4, 8
MWU_PRUNE_KEY_L2SQ, MWU_PRUNE_KEY_L1 = 0, 1
MWU_ALGO_AUTO, MWU_ALGO_ONE_PASS, MWU_ALGO_MULTI_PASS = 0, 1, 2


class MwuError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class ProjDesc(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("block", ctypes.c_int32),
                ("prune_key", ctypes.c_int32), ("k_unify", ctypes.c_int64),
                ("k_prune", ctypes.c_int64), ("algo", ctypes.c_int32), ("block_rows", ctypes.c_int32),
                ("prune_group_rows", ctypes.c_int32), ("prune_group_cols", ctypes.c_int32),
                ("block_taps", ctypes.c_int32), ("taps", ctypes.c_int32)]

    @property
    def n_blocks(self) -> int:
        """Blocks of the partition this descriptor names (1-, 2- or 3-dim shape)."""
        dr, dt, taps = max(self.block_rows, 1), max(self.block_taps, 1), max(self.taps, 1)
        return (self.rows // dr) * ((self.cols // taps) // self.block) * ((taps + dt - 1) // dt)


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2106_08301_b200.build` (there is no fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32, i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32, ctypes.c_int64
        dp = ctypes.POINTER(ProjDesc)
        L.mwu_status_string.restype = ctypes.c_char_p
        L.mwu_status_string.argtypes = [ctypes.c_int]
        L.mwu_kernel_launches.restype = ctypes.c_uint64
        L.mwu_kernel_launches.argtypes = []
        L.mwu_count_from_permille.restype = i64
        L.mwu_count_from_permille.argtypes = [i64, i32]
        L.mwu_project_workspace_bytes.restype = sz
        L.mwu_project_workspace_bytes.argtypes = [dp]
        L.mwu_project.restype = ctypes.c_int
        L.mwu_project.argtypes = [dp] + [vp] * 11 + [sz, vp]
        L.mwu_admm_step.restype = ctypes.c_int
        L.mwu_admm_step.argtypes = [dp] + [vp] * 11 + [sz, vp]
        L.mwu_project_static.restype = ctypes.c_int
        L.mwu_project_static.argtypes = [dp] + [vp] * 10 + [vp]
        L.mwu_packed_bytes.restype = sz
        L.mwu_packed_bytes.argtypes = [dp]
        L.mwu_pack.restype = ctypes.c_int
        L.mwu_pack.argtypes = [dp] + [vp] * 7 + [sz, vp, vp]
        L.mwu_gemm.restype = ctypes.c_int
        L.mwu_gemm.argtypes = [dp, vp, vp, i64, i64, vp, i64, i32, vp, vp]
        L.mwu_decode.restype = ctypes.c_int
        L.mwu_decode.argtypes = [dp, vp, vp, i64, vp, vp]
        L.mwu_gemm_workspace_bytes.restype = ctypes.c_size_t
        L.mwu_gemm_workspace_bytes.argtypes = [dp, i64]
        L.mwu_gemm_ws.restype = ctypes.c_int
        L.mwu_gemm_ws.argtypes = [dp, vp, vp, i64, i64, vp, i64, i32, vp, ctypes.c_size_t, vp, vp]
        L.mwu_conv_implicit.restype = ctypes.c_int
        L.mwu_conv_implicit.argtypes = [dp, vp, vp] + [i32] * 8 + [vp, i32, vp, vp]
        L.mwu_conv_workspace_bytes.restype = sz
        L.mwu_conv_workspace_bytes.argtypes = [dp] + [i32] * 8
        L.mwu_conv_implicit_ws.restype = ctypes.c_int
        L.mwu_conv_implicit_ws.argtypes = [dp, vp, vp] + [i32] * 8 + [vp, i32, vp, sz, vp, vp]
        L.mwu_keep_n_of_m.restype = ctypes.c_int
        L.mwu_keep_n_of_m.argtypes = [i64, i64, i32, i32, vp, vp, vp, vp, vp, i64, vp, vp]
        L.mwu_gemm_dense.restype = ctypes.c_int
        L.mwu_gemm_dense.argtypes = [i64, i64, vp, i64, vp, i64, i64, vp, i64, i32, vp, vp]
        L.mwu_conv_dense_workspace_bytes.restype = sz
        L.mwu_conv_dense_workspace_bytes.argtypes = [i64] + [i32] * 8
        L.mwu_conv_dense.restype = ctypes.c_int
        L.mwu_conv_dense.argtypes = [i64, vp, i64, vp] + [i32] * 8 + [vp, i32, vp, sz, vp, vp]
        L.mwu_debug_conv_wait.restype = None
        L.mwu_debug_conv_wait.argtypes = [i64, i64]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def status_string(status: int) -> str:
    return lib().mwu_status_string(int(status)).decode()


def make_desc(rows: int, cols: int, block: int, k_unify: int, k_prune: int,
              prune_key: int = MWU_PRUNE_KEY_L2SQ, algo: int = MWU_ALGO_AUTO,
              prune_group=None, block_rows: int = 0, block_taps: int = 0, taps: int = 0) -> ProjDesc:
    """prune_group = (rows, cols) of a prune group, or None for block-by-block pruning.
    block_rows / block_taps / taps: 2- and 3-dim block shapes (block = channels of a block)."""
    gr, gc = prune_group if prune_group else (0, 0)
    return ProjDesc(int(rows), int(cols), int(block), int(prune_key), int(k_unify), int(k_prune),
                    int(algo), int(block_rows), int(gr), int(gc), int(block_taps), int(taps))


def mwu_kernel_launches() -> int:
    return int(lib().mwu_kernel_launches())


def mwu_count_from_permille(n_blocks: int, permille: int) -> int:
    return int(lib().mwu_count_from_permille(int(n_blocks), int(permille)))


def mwu_project_workspace_bytes(desc: ProjDesc) -> int:
    return int(lib().mwu_project_workspace_bytes(ctypes.byref(desc)))


def mwu_project(desc, W, U_dual, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p,
                dev_status, workspace, stream=None, check=True) -> int:
    rc = lib().mwu_project(ctypes.byref(desc), _ptr(W), _ptr(U_dual), _ptr(Q), _ptr(u),
                           _ptr(pruned_bitmap), _ptr(unified_bitmap), _ptr(sign_bits),
                           _ptr(loss_u), _ptr(loss_p), _ptr(dev_status), _ptr(workspace),
                           workspace.numel() * workspace.element_size() if workspace is not None else 0,
                           _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_project")
    return rc


def mwu_admm_step(desc, W, U_dual, Q, U_next, residual_sq, u, pruned_bitmap, unified_bitmap, sign_bits,
                  dev_status, workspace, stream=None, check=True) -> int:
    """Projection plus dual update U_next = V - Q and residual_sq = ||V - Q||_F^2 in one call."""
    rc = lib().mwu_admm_step(ctypes.byref(desc), _ptr(W), _ptr(U_dual), _ptr(Q), _ptr(U_next),
                             _ptr(residual_sq), _ptr(u), _ptr(pruned_bitmap), _ptr(unified_bitmap),
                             _ptr(sign_bits), _ptr(dev_status), _ptr(workspace),
                             workspace.numel() * workspace.element_size() if workspace is not None else 0,
                             _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_admm_step")
    return rc


def mwu_project_static(desc, W, U_dual, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u,
                       loss_p, dev_status, stream=None, check=True) -> int:
    """mwu_project on the library's built-in scratch: no workspace argument, no allocation."""
    rc = lib().mwu_project_static(ctypes.byref(desc), _ptr(W), _ptr(U_dual), _ptr(Q), _ptr(u),
                                  _ptr(pruned_bitmap), _ptr(unified_bitmap), _ptr(sign_bits),
                                  _ptr(loss_u), _ptr(loss_p), _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_project_static")
    return rc


def mwu_packed_bytes(desc: ProjDesc) -> int:
    return int(lib().mwu_packed_bytes(ctypes.byref(desc)))


def mwu_pack(desc, W, U_dual, u, pruned_bitmap, unified_bitmap, sign_bits, packed, dev_status,
             stream=None, check=True) -> int:
    rc = lib().mwu_pack(ctypes.byref(desc), _ptr(W), _ptr(U_dual), _ptr(u), _ptr(pruned_bitmap),
                        _ptr(unified_bitmap), _ptr(sign_bits), _ptr(packed),
                        packed.numel() * packed.element_size() if packed is not None else 0,
                        _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_pack")
    return rc


def mwu_gemm(desc, packed, X, M, ldx, Y, ldy, y_dtype, dev_status, stream=None, check=True) -> int:
    rc = lib().mwu_gemm(ctypes.byref(desc), _ptr(packed), _ptr(X), int(M), int(ldx), _ptr(Y),
                        int(ldy), int(y_dtype), _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_gemm")
    return rc


def mwu_decode(desc, packed, Wd, ldw, dev_status, stream=None, check=True) -> int:
    rc = lib().mwu_decode(ctypes.byref(desc), _ptr(packed), _ptr(Wd), int(ldw), _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_decode")
    return rc


def mwu_gemm_workspace_bytes(desc, M) -> int:
    return int(lib().mwu_gemm_workspace_bytes(ctypes.byref(desc), int(M)))


def mwu_gemm_ws(desc, packed, X, M, ldx, Y, ldy, y_dtype, workspace, dev_status, stream=None, check=True) -> int:
    """mwu_gemm with a scratch tensor (uint8, or None); its size is taken from the tensor."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().mwu_gemm_ws(ctypes.byref(desc), _ptr(packed), _ptr(X), int(M), int(ldx), _ptr(Y), int(ldy),
                           int(y_dtype), _ptr(workspace), nbytes, _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_gemm_ws")
    return rc


def mwu_conv_implicit(desc, packed, X, n, c, h, w, kh, kw, stride, pad, Y, y_dtype, dev_status,
                      stream=None, check=True) -> int:
    rc = lib().mwu_conv_implicit(ctypes.byref(desc), _ptr(packed), _ptr(X), int(n), int(c), int(h),
                                 int(w), int(kh), int(kw), int(stride), int(pad), _ptr(Y),
                                 int(y_dtype), _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_conv_implicit")
    return rc


def mwu_keep_n_of_m(rows, cols, n, m, W, U_dual, Q, keep_bits, Wd, ldw, dev_status, stream=None, check=True) -> int:
    rc = lib().mwu_keep_n_of_m(int(rows), int(cols), int(n), int(m), _ptr(W), _ptr(U_dual), _ptr(Q),
                               _ptr(keep_bits), _ptr(Wd), int(ldw), _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_keep_n_of_m")
    return rc


def mwu_gemm_dense(rows, cols, Wd, ldw, X, M, ldx, Y, ldy, y_dtype, dev_status, stream=None, check=True) -> int:
    rc = lib().mwu_gemm_dense(int(rows), int(cols), _ptr(Wd), int(ldw), _ptr(X), int(M), int(ldx), _ptr(Y),
                              int(ldy), int(y_dtype), _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_gemm_dense")
    return rc


def mwu_conv_dense_workspace_bytes(rows, n, c, h, w, kh, kw, stride, pad) -> int:
    return int(lib().mwu_conv_dense_workspace_bytes(int(rows), int(n), int(c), int(h), int(w), int(kh), int(kw),
                                                    int(stride), int(pad)))


def mwu_conv_dense(rows, Wd, ldw, X, n, c, h, w, kh, kw, stride, pad, Y, y_dtype, workspace, dev_status,
                   stream=None, check=True) -> int:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().mwu_conv_dense(int(rows), _ptr(Wd), int(ldw), _ptr(X), int(n), int(c), int(h), int(w), int(kh),
                              int(kw), int(stride), int(pad), _ptr(Y), int(y_dtype), _ptr(workspace), nbytes,
                              _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_conv_dense")
    return rc


def mwu_debug_conv_wait(limit_cycles: int, withhold_stage: int) -> None:
    lib().mwu_debug_conv_wait(int(limit_cycles), int(withhold_stage))


def mwu_conv_workspace_bytes(desc, n, c, h, w, kh, kw, stride, pad) -> int:
    return int(lib().mwu_conv_workspace_bytes(ctypes.byref(desc), int(n), int(c), int(h), int(w), int(kh),
                                              int(kw), int(stride), int(pad)))


def mwu_conv_implicit_ws(desc, packed, X, n, c, h, w, kh, kw, stride, pad, Y, y_dtype, workspace, dev_status,
                         stream=None, check=True) -> int:
    """mwu_conv_implicit with a scratch tensor (uint8, or None); its size is taken from the tensor."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().mwu_conv_implicit_ws(ctypes.byref(desc), _ptr(packed), _ptr(X), int(n), int(c), int(h),
                                    int(w), int(kh), int(kw), int(stride), int(pad), _ptr(Y),
                                    int(y_dtype), _ptr(workspace), nbytes, _ptr(dev_status), _stream(stream))
    if check and rc != MWU_OK:
        raise MwuError(rc, "mwu_conv_implicit_ws")
    return rc


# ------------------------------------------------------------------------------------------
# convenience: allocate the outputs of a projection (torch is used for device memory only)
# ------------------------------------------------------------------------------------------
class ProjectionBuffers:
    """Device buffers for one mwu_project call on a [rows, cols] weight."""

    def __init__(self, desc: ProjDesc, device="cuda", want_q=True, want_loss=False):
        mb = desc.n_blocks
        n = desc.rows * desc.cols
        self.desc = desc
        self.Q = torch.empty(n, dtype=torch.float32, device=device) if want_q else None
        self.u = torch.empty(mb, dtype=torch.float32, device=device)
        self.pruned_bitmap = torch.empty((mb + 31) // 32, dtype=torch.int32, device=device)
        self.unified_bitmap = torch.empty((mb + 31) // 32, dtype=torch.int32, device=device)
        self.sign_bits = torch.empty((n + 31) // 32, dtype=torch.int32, device=device)
        self.loss_u = torch.empty(mb, dtype=torch.float64, device=device) if want_loss else None
        self.loss_p = torch.empty(mb, dtype=torch.float64, device=device) if want_loss else None
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)
        self.workspace = torch.empty(mwu_project_workspace_bytes(desc), dtype=torch.uint8,
                                     device=device)

    def project(self, W, U_dual=None, stream=None):
        return mwu_project(self.desc, W, U_dual, self.Q, self.u, self.pruned_bitmap,
                           self.unified_bitmap, self.sign_bits, self.loss_u, self.loss_p,
                           self.dev_status, self.workspace, stream)

    def admm_step(self, W, U_dual, U_next, residual_sq, stream=None):
        return mwu_admm_step(self.desc, W, U_dual, self.Q, U_next, residual_sq, self.u,
                             self.pruned_bitmap, self.unified_bitmap, self.sign_bits,
                             self.dev_status, self.workspace, stream)

    def pack(self, W, U_dual=None, packed=None, stream=None):
        if packed is None:
            packed = torch.empty(mwu_packed_bytes(self.desc), dtype=torch.uint8, device=W.device)
        mwu_pack(self.desc, W, U_dual, self.u, self.pruned_bitmap, self.unified_bitmap,
                 self.sign_bits, packed, self.dev_status, stream)
        return packed
