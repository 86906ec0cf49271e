"""ctypes binding of librazer.so: the C entry points of include/razer.h, one to one.

Argument marshalling only: tensors are passed as raw device (or host) pointers, the
current torch CUDA stream as the stream argument.  Every computation runs in the
library's CUDA kernels; there is no CPU fallback.  Importing this module loads the
library and raises if it has not been built (python -m paper_2501_04052_b200.build).
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("RAZER_LIB") or os.path.join(_HERE, "librazer.so")   # RAZER_LIB: load another build of the library

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT = -1, -2, -3, -4, -5
SCALE_E3M3_META2, SCALE_E4M3_META1 = 0, 1
OP_GEMV, OP_GEMM, OP_GEMM_W4A4 = 0, 1, 2

EXPORTS = (
    "razer_last_error", "razer_version", "razer_kernel_launches", "razer_packed_bytes", "razer_pack_layout", "razer_dequant",
    "razer_workspace_bytes", "razer_workspace_init", "razer_workspace_status", "razer_gemv", "razer_gemm", "razer_gemv_host", "razer_quant_act",
    "razer_decode_act", "razer_gemm_w4a4", "razer_gemv_static", "razer_quant_weight",
    "razer_fp4_act_bytes", "razer_quant_act_fp4", "razer_gemm_w4a4_fp4",
)


class RazerDesc(ctypes.Structure):
    """Mirror of `razer_desc` in include/razer.h."""
    _fields_ = [("N", c_int32), ("K", c_int32), ("block", c_int32), ("scale_fmt", c_int32),
                ("remap_code", c_int32), ("sv_mag", c_float * 2), ("tensor_scale", c_float)]


class RazerError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"razer error {code}: {msg}")
        self.code = code


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2501_04052_b200.build`; "
                      "there is no fallback path")
_lib = ctypes.CDLL(LIB_PATH)

_lib.razer_last_error.restype = c_char_p
_lib.razer_last_error.argtypes = []
_lib.razer_version.restype = c_int
_lib.razer_packed_bytes.argtypes = [POINTER(RazerDesc), POINTER(c_size_t)]
_lib.razer_pack_layout.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_void_p, c_void_p]
_lib.razer_dequant.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_int, c_void_p]
_lib.razer_workspace_bytes.argtypes = [POINTER(RazerDesc), c_int, c_int, POINTER(c_size_t)]
_lib.razer_workspace_init.argtypes = [c_void_p, c_size_t, c_void_p]
_lib.razer_workspace_status.argtypes = [c_void_p, c_void_p]
_lib.razer_gemv.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_size_t, c_void_p]
_lib.razer_gemm.argtypes = _lib.razer_gemv.argtypes
_lib.razer_gemv_host.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                 c_void_p, c_size_t, c_void_p]
_lib.razer_gemv_static.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_int, c_void_p, c_void_p]
_lib.razer_quant_act.argtypes = [c_void_p, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p, c_void_p,
                                 c_void_p, c_void_p]
_lib.razer_quant_weight.argtypes = [c_void_p, c_int, c_int, c_int, c_int, POINTER(c_float), c_int, c_void_p, c_void_p, c_void_p,
                                    c_void_p, c_void_p, c_void_p]
_lib.razer_fp4_act_bytes.argtypes = [c_int, c_int, POINTER(c_size_t)]
_lib.razer_quant_act_fp4.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
_lib.razer_gemm_w4a4_fp4.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_size_t,
                                     c_void_p]
_lib.razer_decode_act.argtypes = [c_void_p, c_void_p, c_int, c_int, c_float, c_void_p, c_void_p]
_lib.razer_gemm_w4a4.argtypes = [POINTER(RazerDesc), c_void_p, c_void_p, c_void_p, c_void_p, c_float, c_int,
                                 c_void_p, c_void_p, c_size_t, c_int, c_void_p]
for _n in EXPORTS:
    if _n not in ("razer_last_error", "razer_kernel_launches"):
        getattr(_lib, _n).restype = c_int
_lib.razer_kernel_launches.restype = ctypes.c_ulonglong
_lib.razer_kernel_launches.argtypes = []


def lib() -> ctypes.CDLL:
    return _lib


def last_error() -> str:
    return _lib.razer_last_error().decode()


def _check(rc: int) -> None:
    if rc != OK:
        raise RazerError(rc, last_error())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def make_desc(N: int, K: int, tensor_scale: float, sv_mag=(5.0, 8.0), remap_code: int = 0x8,
              block: int = 16, scale_fmt: int = SCALE_E3M3_META2) -> RazerDesc:
    d = RazerDesc()
    d.N, d.K, d.block, d.scale_fmt, d.remap_code = N, K, block, scale_fmt, remap_code
    d.sv_mag[0], d.sv_mag[1] = float(sv_mag[0]), float(sv_mag[1])
    d.tensor_scale = float(tensor_scale)
    return d


def razer_version() -> int:
    return _lib.razer_version()


def razer_kernel_launches() -> int:
    return int(_lib.razer_kernel_launches())


def razer_packed_bytes(desc: RazerDesc) -> int:
    n = c_size_t(0)
    _check(_lib.razer_packed_bytes(ctypes.byref(desc), ctypes.byref(n)))
    return n.value


def razer_workspace_bytes(desc: RazerDesc, M: int, op: int) -> int:
    n = c_size_t(0)
    _check(_lib.razer_workspace_bytes(ctypes.byref(desc), M, op, ctypes.byref(n)))
    return n.value


def razer_pack_layout(desc: RazerDesc, codes: torch.Tensor, scales: torch.Tensor,
                      packed: torch.Tensor | None = None) -> torch.Tensor:
    """codes uint8 [N, K/2], scales uint8 [N, K/16] (device) -> packed uint8 buffer (device)."""
    assert codes.is_cuda and scales.is_cuda and codes.is_contiguous() and scales.is_contiguous()
    if packed is None:
        packed = torch.empty(razer_packed_bytes(desc), dtype=torch.uint8, device=codes.device)
    _check(_lib.razer_pack_layout(ctypes.byref(desc), _ptr(codes), _ptr(scales), _ptr(packed), _stream()))
    return packed


def razer_dequant(desc: RazerDesc, packed: torch.Tensor, fp32: bool) -> torch.Tensor:
    out = torch.empty((desc.N, desc.K), dtype=torch.float32 if fp32 else torch.bfloat16, device=packed.device)
    _check(_lib.razer_dequant(ctypes.byref(desc), _ptr(packed), _ptr(out), 1 if fp32 else 0, _stream()))
    return out


def razer_workspace_init(workspace: torch.Tensor) -> None:
    _check(_lib.razer_workspace_init(_ptr(workspace), workspace.numel(), _stream()))


def razer_workspace_status(workspace: torch.Tensor) -> None:
    """Synchronizes the stream; raises RazerError(ERR_DEVICE_TIMEOUT) if a kernel gave up a wait."""
    _check(_lib.razer_workspace_status(_ptr(workspace), _stream()))


def alloc_workspace(desc: RazerDesc, M: int, op: int, device) -> torch.Tensor:
    """Allocate (torch) and prepare (razer_workspace_init) a workspace for `op` with M rows."""
    n = razer_workspace_bytes(desc, M, op)
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device=device)
    razer_workspace_init(ws)
    return ws


def _matmul(fn, desc, packed, x, y, workspace, op):
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.shape[1] == desc.K
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, desc.N), dtype=torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(desc, M, op, x.device)
    _check(fn(ctypes.byref(desc), _ptr(packed), _ptr(x), M, _ptr(y), _ptr(workspace), workspace.numel(), _stream()))
    return y


def razer_gemv(desc, packed, x, y=None, workspace=None) -> torch.Tensor:
    """x bf16 [M, K] (M <= 64, device) -> y bf16 [M, N]."""
    return _matmul(_lib.razer_gemv, desc, packed, x, y, workspace, OP_GEMV)


def razer_gemm(desc, packed, x, y=None, workspace=None) -> torch.Tensor:
    """x bf16 [M, K] (device) -> y bf16 [M, N]."""
    return _matmul(_lib.razer_gemm, desc, packed, x, y, workspace, OP_GEMM)


def razer_gemv_static(desc, packed, x, y) -> torch.Tensor:
    """razer_gemv without a workspace argument: the library's built-in scratch array is used, so
    nothing is allocated here either (the caller brings y).  x bf16 [M, K] with M <= 16."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.shape[1] == desc.K
    assert y.is_cuda and y.dtype == torch.bfloat16 and y.is_contiguous() and tuple(y.shape) == (x.shape[0], desc.N)
    _check(_lib.razer_gemv_static(ctypes.byref(desc), _ptr(packed), _ptr(x), x.shape[0], _ptr(y), _stream()))
    return y


def razer_gemv_host(desc, packed, x_host, y_host, x_stage, y_stage, workspace) -> None:
    """x_host / y_host: pinned CPU bf16 tensors; x_stage / y_stage / workspace: device buffers."""
    assert not x_host.is_cuda and not y_host.is_cuda
    M = x_host.shape[0]
    _check(_lib.razer_gemv_host(ctypes.byref(desc), _ptr(packed), _ptr(x_host), M, _ptr(y_host), _ptr(x_stage),
                                _ptr(y_stage), _ptr(workspace), workspace.numel(), _stream()))


_quant_act_scratch = {}


def razer_quant_act(x: torch.Tensor, sv_mag: float = 5.0, tensor_scale: torch.Tensor | None = None,
                    scratch: torch.Tensor | None = None):
    """x bf16 [M, K] (device) -> (codes uint8 [M, K/2], scales uint8 [M, K/16], tensor scale float32 [1]).
    `scratch`: two zeroed int32 on the device (left zero by every call); one per device is kept here when none is given."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    M, K = x.shape
    codes = torch.empty((M, K // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty((M, K // 16), dtype=torch.uint8, device=x.device)
    out_scale = torch.empty(1, dtype=torch.float32, device=x.device)
    if scratch is None:
        scratch = _quant_act_scratch.get(x.device)
        if scratch is None:
            scratch = _quant_act_scratch[x.device] = torch.zeros(2, dtype=torch.int32, device=x.device)
    _check(_lib.razer_quant_act(_ptr(x), M, K, float(sv_mag), _ptr(tensor_scale), _ptr(scratch), _ptr(codes),
                                _ptr(scales), _ptr(out_scale), _stream()))
    return codes, scales, out_scale


def razer_quant_weight(w: torch.Tensor, sv_mag=(5.0, 8.0), remap_code: int = 0x8,
                       tensor_scale: torch.Tensor | None = None, block: int = 16, scale_aware: bool = False):
    """w FP32 [N, K] (device) -> (codes uint8 [N, K/2], scales uint8 [N, K/block], tensor scale float32 [1]) in the
    interchange format that razer_pack_layout reads."""
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
    N, K = w.shape
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=w.device)
    scales = torch.empty((N, K // block), dtype=torch.uint8, device=w.device)
    out_scale = torch.empty(1, dtype=torch.float32, device=w.device)
    scratch = torch.empty(1, dtype=torch.int32, device=w.device)
    mags = (c_float * 2)(float(sv_mag[0]), float(sv_mag[1]))
    _check(_lib.razer_quant_weight(_ptr(w), N, K, int(block), int(bool(scale_aware)), mags, int(remap_code), _ptr(tensor_scale), _ptr(scratch),
                                   _ptr(codes), _ptr(scales), _ptr(out_scale), _stream()))
    return codes, scales, out_scale


def razer_fp4_act_bytes(M: int, K: int) -> int:
    n = c_size_t()
    _check(_lib.razer_fp4_act_bytes(int(M), int(K), ctypes.byref(n)))
    return n.value


def razer_quant_act_fp4(x: torch.Tensor, tensor_scale: torch.Tensor | None = None, act_fp4: torch.Tensor | None = None,
                        scratch: torch.Tensor | None = None):
    """x bf16 [M, K] (device) -> (FP4 activation operand of the block-scaled kernel uint8 [bytes], tensor scale float32 [1])."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    M, K = x.shape
    if act_fp4 is None:
        act_fp4 = torch.empty(razer_fp4_act_bytes(M, K), dtype=torch.uint8, device=x.device)
    out_scale = torch.empty(1, dtype=torch.float32, device=x.device)
    if scratch is None:
        scratch = _quant_act_scratch.get(x.device)
        if scratch is None:
            scratch = _quant_act_scratch[x.device] = torch.zeros(2, dtype=torch.int32, device=x.device)
    _check(_lib.razer_quant_act_fp4(_ptr(x), M, K, _ptr(tensor_scale), _ptr(scratch), _ptr(act_fp4), _ptr(out_scale),
                                    _stream()))
    return act_fp4, out_scale


def razer_gemm_w4a4_fp4(desc, packed, act_fp4, act_tensor_scale, M: int, y=None, workspace=None) -> torch.Tensor:
    if y is None:
        y = torch.empty((M, desc.N), dtype=torch.bfloat16, device=act_fp4.device)
    if workspace is None:
        workspace = alloc_workspace(desc, M, OP_GEMM_W4A4, act_fp4.device)
    _check(_lib.razer_gemm_w4a4_fp4(ctypes.byref(desc), _ptr(packed), _ptr(act_fp4), _ptr(act_tensor_scale), int(M), _ptr(y),
                                    _ptr(workspace), workspace.numel(), _stream()))
    return y


def razer_decode_act(codes: torch.Tensor, scales: torch.Tensor, sv_mag: float = 5.0) -> torch.Tensor:
    M, K = codes.shape[0], codes.shape[1] * 2
    out = torch.empty((M, K), dtype=torch.bfloat16, device=codes.device)
    _check(_lib.razer_decode_act(_ptr(codes), _ptr(scales), M, K, float(sv_mag), _ptr(out), _stream()))
    return out


def razer_gemm_w4a4(desc, packed, act_codes, act_scales, act_tensor_scale, act_sv_mag: float = 5.0, y=None,
                    workspace=None, use_native_fp4: bool = False) -> torch.Tensor:
    M = act_codes.shape[0]
    if y is None:
        y = torch.empty((M, desc.N), dtype=torch.bfloat16, device=act_codes.device)
    if workspace is None:
        workspace = alloc_workspace(desc, M, OP_GEMM_W4A4, act_codes.device)
    _check(_lib.razer_gemm_w4a4(ctypes.byref(desc), _ptr(packed), _ptr(act_codes), _ptr(act_scales),
                                _ptr(act_tensor_scale), float(act_sv_mag), M, _ptr(y), _ptr(workspace),
                                workspace.numel(), 1 if use_native_fp4 else 0, _stream()))
    return y
