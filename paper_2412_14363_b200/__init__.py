"""Python binding of libresq.so (the ResQ mixed-precision linear layer for B200).

Argument marshalling only: every function takes torch CUDA tensors (used purely as device buffers),
passes their addresses and the current CUDA stream to the C entry point of the same name, and raises
`ResqError` on a non-zero status.  There is no fallback: if the shared library is missing the import
fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libresq.so")

OK, ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT, ERR_INDEX = range(9)
SCALE_FP32, SCALE_FP16 = 0, 1
OPT_DECODE_EARLY_WEIGHTS, OPT_WAIT_LIMIT_US = 1, 2
Y_BF16, Y_FP32 = 0, 1

EXPORTS = [
    "resq_w8_bytes", "resq_w4_bytes", "resq_w4_i8_bytes", "resq_scale_bytes", "resq_workspace_bytes",
    "resq_pack_weights", "resq_pack_weights_gptq", "resq_pack_weights_projected", "resq_pack_projected_workspace_bytes", "resq_project", "resq_project_workspace_bytes", "resq_hadamard_quantize", "resq_project_quantize", "resq_project_quantize_static", "resq_mixed_gemm", "resq_linear",
    "resq_unpack_int4", "resq_set_option",
    "resq_weight_row_sums", "resq_project_quantize_asym", "resq_mixed_gemm_asym", "resq_linear_asym",
    "resq_workspace_bytes_asym",
    "resq_device_status", "resq_launch_count", "resq_selftest_wait_runs_out", "resq_status_string", "resq_last_cuda_error",
]


class ResqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = f": {lib.resq_last_cuda_error().decode()}" if status == ERR_CUDA else ""
        super().__init__(f"{where}: status {status} ({status_string(status)}{detail})")


class LayerDesc(ctypes.Structure):
    _fields_ = [("K", ctypes.c_int32), ("n_out", ctypes.c_int32), ("r", ctypes.c_int32),
                ("w_scale_dtype", ctypes.c_int32)]


class WeightsStruct(ctypes.Structure):
    _fields_ = [("w8", ctypes.c_void_p), ("w4", ctypes.c_void_p), ("s_w8", ctypes.c_void_p),
                ("s_w4", ctypes.c_void_p), ("w4_i8", ctypes.c_void_p)]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} not found: build it with `python __graft_entry__.py` "
                      "(there is no CPU or PyTorch fallback)")
lib = ctypes.CDLL(LIB_PATH)

_vp, _sz, _i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_dp = ctypes.POINTER(LayerDesc)
for _n in ("resq_w8_bytes", "resq_w4_bytes", "resq_w4_i8_bytes", "resq_scale_bytes"):
    getattr(lib, _n).restype = _sz
    getattr(lib, _n).argtypes = [_dp]
lib.resq_workspace_bytes.restype = _sz
lib.resq_workspace_bytes.argtypes = [_dp, _i, _i, _i]
lib.resq_pack_weights.argtypes = [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.resq_pack_weights_gptq.argtypes = [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.resq_pack_projected_workspace_bytes.restype = _sz
lib.resq_pack_projected_workspace_bytes.argtypes = [_dp]
lib.resq_pack_weights_projected.argtypes = [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.resq_project.argtypes = [_vp, _vp, _i, _i, _vp, _vp, _sz, _vp]
lib.resq_project_workspace_bytes.restype = _sz
lib.resq_project_workspace_bytes.argtypes = []
lib.resq_hadamard_quantize.argtypes = [_vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
lib.resq_project_quantize.argtypes = [_vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.resq_project_quantize_static.argtypes = [_vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
lib.resq_mixed_gemm.argtypes = [_dp, _i, _vp, _vp, _vp, _vp, _vp, ctypes.POINTER(WeightsStruct), _vp, _i, _vp, _vp,
                                _vp, _sz, _vp]
lib.resq_linear.argtypes = [_dp, _i, _vp, _vp, ctypes.POINTER(WeightsStruct), _vp, _i, _vp, _sz, _vp]
lib.resq_unpack_int4.argtypes = [_vp, _vp, _sz, _sz, _vp]
lib.resq_weight_row_sums.argtypes = [_dp, ctypes.POINTER(WeightsStruct), _vp, _vp, _vp]
lib.resq_project_quantize_asym.argtypes = [_vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.resq_mixed_gemm_asym.argtypes = [_dp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.POINTER(WeightsStruct), _vp, _vp,
                                     _vp, _i, _vp, _vp, _vp, _sz, _vp]
lib.resq_linear_asym.argtypes = [_dp, _i, _vp, _vp, ctypes.POINTER(WeightsStruct), _vp, _vp, _vp, _i, _vp, _sz, _vp]
lib.resq_workspace_bytes_asym.restype = _sz
lib.resq_workspace_bytes_asym.argtypes = [_dp, _i, _i, _i]
lib.resq_set_option.argtypes = [_i, _i]
lib.resq_device_status.argtypes = [_vp]
lib.resq_selftest_wait_runs_out.argtypes = [_vp]
lib.resq_launch_count.restype = ctypes.c_ulonglong
lib.resq_launch_count.argtypes = []
lib.resq_status_string.restype = ctypes.c_char_p
lib.resq_last_cuda_error.restype = ctypes.c_char_p
lib.resq_last_cuda_error.argtypes = []
lib.resq_status_string.argtypes = [_i]


def status_string(status: int) -> str:
    return lib.resq_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != OK:
        raise ResqError(status, where)


def layer_desc(K: int, n_out: int, r: int, w_scale_dtype: int = SCALE_FP32) -> LayerDesc:
    return LayerDesc(K, n_out, r, w_scale_dtype)


def resq_workspace_bytes(desc: LayerDesc, T: int, has_P: bool, has_w4_i8: bool) -> int:
    return int(lib.resq_workspace_bytes(ctypes.byref(desc), T, int(has_P), int(has_w4_i8)))


@dataclass
class Weights:
    """Device buffers written by resq_pack_weights (torch tensors as storage)."""
    desc: LayerDesc
    w8: object
    w4: object
    s_w8: object
    s_w4: object
    w4_i8: object = None

    def struct(self) -> WeightsStruct:
        return WeightsStruct(_ptr(self.w8), _ptr(self.w4), _ptr(self.s_w8), _ptr(self.s_w4), _ptr(self.w4_i8))


def resq_pack_weights(desc: LayerDesc, W_proj, with_w4_i8: bool = True) -> Weights:
    """W_proj: float32 CUDA tensor [n_out][K].  Allocates the packed buffers and fills them."""
    import torch
    assert W_proj.is_cuda and W_proj.dtype == torch.float32 and W_proj.is_contiguous()
    assert tuple(W_proj.shape) == (desc.n_out, desc.K)
    dev = W_proj.device
    K4 = desc.K - desc.r
    sdt = torch.float16 if desc.w_scale_dtype == SCALE_FP16 else torch.float32
    w = Weights(desc,
                torch.empty((desc.n_out, desc.r), dtype=torch.int8, device=dev),
                torch.empty((desc.n_out, K4 // 2), dtype=torch.uint8, device=dev),
                torch.empty(desc.n_out, dtype=sdt, device=dev),
                torch.empty(desc.n_out, dtype=sdt, device=dev),
                torch.empty((desc.n_out, K4), dtype=torch.int8, device=dev) if with_w4_i8 else None)
    _check(lib.resq_pack_weights(ctypes.byref(desc), _ptr(W_proj), _ptr(w.w8), _ptr(w.w4), _ptr(w.s_w8),
                                 _ptr(w.s_w4), _ptr(w.w4_i8), _stream()), "resq_pack_weights")
    return w


def resq_pack_weights_gptq(desc: LayerDesc, W_proj, U_inv, dead_cols=None, with_w4_i8: bool = True) -> Weights:
    """W_proj fp32 [n_out][K], U_inv fp32 [K][K] (upper Cholesky factor of the inverse Hessian), dead_cols uint8 [K] or
    None: GPTQ rounding instead of round-to-nearest (buffers allocated here)."""
    import torch
    assert W_proj.is_cuda and W_proj.dtype == torch.float32 and tuple(W_proj.shape) == (desc.n_out, desc.K)
    assert U_inv.dtype == torch.float32 and tuple(U_inv.shape) == (desc.K, desc.K) and U_inv.is_contiguous()
    dev = W_proj.device
    K4 = desc.K - desc.r
    sdt = torch.float16 if desc.w_scale_dtype == SCALE_FP16 else torch.float32
    w = Weights(desc,
                torch.empty((desc.n_out, desc.r), dtype=torch.int8, device=dev),
                torch.empty((desc.n_out, K4 // 2), dtype=torch.uint8, device=dev),
                torch.empty(desc.n_out, dtype=sdt, device=dev),
                torch.empty(desc.n_out, dtype=sdt, device=dev),
                torch.empty((desc.n_out, K4), dtype=torch.int8, device=dev) if with_w4_i8 else None)
    _check(lib.resq_pack_weights_gptq(ctypes.byref(desc), _ptr(W_proj), _ptr(U_inv), _ptr(dead_cols), _ptr(w.w8), _ptr(w.w4),
                                      _ptr(w.s_w8), _ptr(w.s_w4), _ptr(w.w4_i8), _stream()), "resq_pack_weights_gptq")
    return w


def resq_pack_weights_projected(desc: LayerDesc, W_raw, U, with_w4_i8: bool = True) -> Weights:
    """W_raw bf16 [n_out][K] (unprojected), U bf16 [K][K]: projects on the GPU and packs (buffers allocated here)."""
    import torch
    assert W_raw.is_cuda and W_raw.dtype == torch.bfloat16 and tuple(W_raw.shape) == (desc.n_out, desc.K)
    assert U.dtype == torch.bfloat16 and tuple(U.shape) == (desc.K, desc.K)
    dev = W_raw.device
    K4 = desc.K - desc.r
    sdt = torch.float16 if desc.w_scale_dtype == SCALE_FP16 else torch.float32
    w = Weights(desc,
                torch.empty((desc.n_out, desc.r), dtype=torch.int8, device=dev),
                torch.empty((desc.n_out, K4 // 2), dtype=torch.uint8, device=dev),
                torch.empty(desc.n_out, dtype=sdt, device=dev),
                torch.empty(desc.n_out, dtype=sdt, device=dev),
                torch.empty((desc.n_out, K4), dtype=torch.int8, device=dev) if with_w4_i8 else None)
    ws = torch.empty(max(int(lib.resq_pack_projected_workspace_bytes(ctypes.byref(desc))), 256), dtype=torch.uint8, device=dev)
    _check(lib.resq_pack_weights_projected(ctypes.byref(desc), _ptr(W_raw), _ptr(U), _ptr(w.w8), _ptr(w.w4), _ptr(w.s_w8),
                                           _ptr(w.s_w4), _ptr(w.w4_i8), _ptr(ws), ws.numel(), _stream()),
           "resq_pack_weights_projected")
    return w


def resq_project_quantize(X, P, r: int, x8, x4, s_x8, s_x4, x4_i8=None, workspace=None):
    """X bf16 [T][K]; P bf16 [K][K] or None; outputs are preallocated CUDA tensors (x4 or x4_i8 may be None)."""
    T, K = X.shape
    _check(lib.resq_project_quantize(_ptr(X), _ptr(P), T, K, r, _ptr(x8), _ptr(x4), _ptr(s_x8), _ptr(s_x4),
                                     _ptr(x4_i8), _ptr(workspace),
                                     0 if workspace is None else workspace.numel() * workspace.element_size(),
                                     _stream()), "resq_project_quantize")


def resq_project(X, P, C, workspace=None):
    """C (fp32 [T][K]) = X (bf16 [T][K]) · P (bf16 [K][K]): the online projection alone.  workspace: optional
    uint8 tensor of resq_project_workspace_bytes() bytes (lets a thin last round of tiles be cut along K)."""
    T, K = X.shape
    _check(lib.resq_project(_ptr(X), _ptr(P), T, K, _ptr(C), _ptr(workspace), _nbytes(workspace), _stream()), "resq_project")


def resq_project_workspace_bytes() -> int:
    return int(lib.resq_project_workspace_bytes())


def resq_hadamard_quantize(X, r: int, x8, x4, s_x8, s_x4, x4_i8=None):
    """X bf16 [T][K] -> codes and scales of X·H_K/sqrt(K) (Hadamard U_D, Section 4.3); r = 0: uniform INT4."""
    T, K = X.shape
    _check(lib.resq_hadamard_quantize(_ptr(X), T, K, r, _ptr(x8), _ptr(x4), _ptr(s_x8), _ptr(s_x4), _ptr(x4_i8),
                                      _stream()), "resq_hadamard_quantize")


STATIC_SCRATCH_BYTES = 8 << 20


def resq_project_quantize_static(X, P, r: int, x8, x4, s_x8, s_x4, x4_i8=None):
    """resq_project_quantize with P given, for callers that cannot allocate a workspace (a process whose
    memory is all owned by another pool, or a loop that must not hit cudaMalloc's device-wide sync):
    the fp32 staging panel is an 8 MiB array inside the library, so T * K * 4 must fit in it.  Calls
    share that array: do not let two of them overlap on the GPU."""
    T, K = X.shape
    _check(lib.resq_project_quantize_static(_ptr(X), _ptr(P), T, K, r, _ptr(x8), _ptr(x4), _ptr(s_x8), _ptr(s_x4),
                                            _ptr(x4_i8), _stream()), "resq_project_quantize_static")


def resq_mixed_gemm(W: Weights, x8, x4, s_x8, s_x4, Y, workspace, dbg_acc8=None, dbg_acc4=None, x4_i8=None):
    import torch
    T = s_x8.shape[0]  # x8 may be None for a uniform INT4 layer (r = 0)
    y_dtype = Y_BF16 if Y.dtype == torch.bfloat16 else Y_FP32
    ws = W.struct()
    _check(lib.resq_mixed_gemm(ctypes.byref(W.desc), T, _ptr(x8), _ptr(x4), _ptr(x4_i8), _ptr(s_x8), _ptr(s_x4),
                               ctypes.byref(ws), _ptr(Y), y_dtype, _ptr(dbg_acc8), _ptr(dbg_acc4), _ptr(workspace),
                               0 if workspace is None else workspace.numel() * workspace.element_size(),
                               _stream()), "resq_mixed_gemm")


def resq_linear(W: Weights, X, P, Y, workspace):
    import torch
    T = X.shape[0]
    y_dtype = Y_BF16 if Y.dtype == torch.bfloat16 else Y_FP32
    ws = W.struct()
    _check(lib.resq_linear(ctypes.byref(W.desc), T, _ptr(X), _ptr(P), ctypes.byref(ws), _ptr(Y), y_dtype,
                           _ptr(workspace),
                           0 if workspace is None else workspace.numel() * workspace.element_size(), _stream()),
           "resq_linear")


def resq_unpack_int4(packed, out):
    rows, half = packed.shape
    _check(lib.resq_unpack_int4(_ptr(packed), _ptr(out), rows, half * 2, _stream()), "resq_unpack_int4")


def resq_set_option(option: int, value: int):
    _check(lib.resq_set_option(int(option), int(value)), "resq_set_option")


def resq_device_status() -> int:
    return int(lib.resq_device_status(_stream()))


def resq_launch_count() -> int:
    """Kernels enqueued by the library in this process so far."""
    return int(lib.resq_launch_count())


def resq_selftest_wait_runs_out():
    """Enqueues the kernel whose bounded wait runs out (see resq.h); resq_device_status then reads ERR_TIMEOUT."""
    _check(lib.resq_selftest_wait_runs_out(_stream()), "resq_selftest_wait_runs_out")


def alloc_workspace(desc: LayerDesc, T: int, has_P: bool, has_w4_i8: bool, device="cuda"):
    import torch
    n = resq_workspace_bytes(desc, T, has_P, has_w4_i8)
    return torch.empty(max(n, 256), dtype=torch.uint8, device=device)


# --------------------------------------------------------------------------- asymmetric activations
def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def resq_weight_row_sums(W: Weights):
    """int32 row sums of the INT8 and INT4 weight codes of a packed layer: (wsum8 [n_out], wsum4 [n_out])."""
    import torch
    dev = W.w8.device
    s8 = torch.empty(W.desc.n_out, dtype=torch.int32, device=dev)
    s4 = torch.empty(W.desc.n_out, dtype=torch.int32, device=dev)
    ws = W.struct()
    _check(lib.resq_weight_row_sums(ctypes.byref(W.desc), ctypes.byref(ws), _ptr(s8), _ptr(s4), _stream()),
           "resq_weight_row_sums")
    return s8, s4


def resq_project_quantize_asym(X, P, r: int, u8, u4, s_x8, s_x4, z_x8, z_x4, u4_u8=None, workspace=None):
    T, K = X.shape
    _check(lib.resq_project_quantize_asym(_ptr(X), _ptr(P), T, K, r, _ptr(u8), _ptr(u4), _ptr(s_x8), _ptr(s_x4),
                                          _ptr(z_x8), _ptr(z_x4), _ptr(u4_u8), _ptr(workspace), _nbytes(workspace),
                                          _stream()), "resq_project_quantize_asym")


def resq_mixed_gemm_asym(W: Weights, wsum8, wsum4, u8, u4, s_x8, s_x4, z_x8, z_x4, Y, workspace, dbg_acc8=None,
                         dbg_acc4=None, u4_u8=None):
    import torch
    T = s_x8.shape[0]
    y_dtype = Y_BF16 if Y.dtype == torch.bfloat16 else Y_FP32
    ws = W.struct()
    _check(lib.resq_mixed_gemm_asym(ctypes.byref(W.desc), T, _ptr(u8), _ptr(u4), _ptr(u4_u8), _ptr(s_x8), _ptr(s_x4),
                                    _ptr(z_x8), _ptr(z_x4), ctypes.byref(ws), _ptr(wsum8), _ptr(wsum4), _ptr(Y), y_dtype,
                                    _ptr(dbg_acc8), _ptr(dbg_acc4), _ptr(workspace), _nbytes(workspace), _stream()),
           "resq_mixed_gemm_asym")


def resq_linear_asym(W: Weights, wsum8, wsum4, X, P, Y, workspace):
    import torch
    T = X.shape[0]
    y_dtype = Y_BF16 if Y.dtype == torch.bfloat16 else Y_FP32
    ws = W.struct()
    _check(lib.resq_linear_asym(ctypes.byref(W.desc), T, _ptr(X), _ptr(P), ctypes.byref(ws), _ptr(wsum8), _ptr(wsum4),
                                _ptr(Y), y_dtype, _ptr(workspace), _nbytes(workspace), _stream()), "resq_linear_asym")


def alloc_workspace_asym(desc: LayerDesc, T: int, has_P: bool, has_w4_i8: bool, device="cuda"):
    import torch
    n = int(lib.resq_workspace_bytes_asym(ctypes.byref(desc), T, int(has_P), int(has_w4_i8)))
    return torch.empty(max(n, 256), dtype=torch.uint8, device=device)
