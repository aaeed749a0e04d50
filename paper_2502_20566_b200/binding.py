"""ctypes binding of ``libsradamw.so`` with the same names as the C ABI (see ``include/sradamw.h``).

Argument marshalling only: every step of the update runs in the library's CUDA kernels.  Tensors
are torch CUDA tensors (used for device memory and streams); BF16 tensors are passed by address.
There is no CPU fallback: a missing library or a failing call raises.
"""

from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_double, c_float, c_int, c_size_t, c_uint16, c_uint32, c_uint64, c_void_p
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsradamw.so")

SR_OK, SR_ERR_INVALID_ARG, SR_ERR_UNSUPPORTED_DEVICE, SR_ERR_WORKSPACE, SR_ERR_CUDA = range(5)
SR_DT_BF16, SR_DT_F32 = 0, 1
SR_FLAG_SR_P, SR_FLAG_SR_M, SR_FLAG_SR_V = 1, 2, 4
SR_FLAGS_DEFAULT = 7
SR_FLAG_EPS_INSIDE = 8

EXPORTS = (
    "sr_downcast_f32_bf16", "sr_downcast_f32_fp8", "sr_downcast_f32_fp4", "sr_accumulate_bf16", "sr_adamw_step", "sr_adamw_step_launch_count", "sr_master_adamw_step", "sr_adamw_step_host", "sr_adamw_step_host_staging_bytes",
    "sr_mt_plan_create", "sr_adamw_multi_tensor",
    "sr_mt_plan_destroy", "sr_mt_plan_total_elements", "grad_sqnorm_workspace_bytes", "grad_sqnorm",
    "grad_sqnorm_static", "grad_sqnorm_static_max_elements", "grad_sqnorm_multi_tensor", "grad_sqnorm_multi_tensor_workspace_bytes",
    "sr_clip_scale", "sr_selftest_in_range_arithmetic", "sr_status_string", "sr_last_cuda_error", "sr_abi_version",
)


class SrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().sr_status_string(status).decode()
        if status == SR_ERR_CUDA:
            msg += f" [cudaError {lib().sr_last_cuda_error()}]"
        super().__init__(f"{where}: {msg}")


class HParams(ctypes.Structure):
    """Mirror of ``sr_adamw_hparams``."""
    _fields_ = [
        ("struct_size", c_uint32),
        ("lr", c_float),
        ("beta1", c_float),
        ("beta2", c_float),
        ("eps", c_float),
        ("weight_decay", c_float),
        ("grad_scale", c_float),
        ("grad_scale_dev", c_void_p),
        ("flags", c_uint32),
    ]


def hparams(lr: float, beta1: float, beta2: float, eps: float, weight_decay: float, grad_scale: float = 1.0,
            grad_scale_dev: Optional[torch.Tensor] = None, flags: int = SR_FLAGS_DEFAULT) -> HParams:
    if grad_scale_dev is not None:
        _want(grad_scale_dev, torch.float32, "grad_scale_dev")
    return HParams(ctypes.sizeof(HParams), lr, beta1, beta2, eps, weight_decay, grad_scale,
                   grad_scale_dev.data_ptr() if grad_scale_dev is not None else None, flags)


_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2502_20566_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.sr_downcast_f32_bf16.argtypes = [c_void_p, c_void_p, c_uint64, c_uint64, c_uint32, c_uint32, c_uint64, c_void_p]
        L.sr_downcast_f32_bf16.restype = c_int
        L.sr_downcast_f32_fp8.argtypes = [c_void_p, c_void_p, c_uint64, c_int, c_uint64, c_uint32, c_uint32, c_uint64, c_void_p]
        L.sr_downcast_f32_fp8.restype = c_int
        L.sr_downcast_f32_fp4.argtypes = [c_void_p, c_void_p, c_uint64, c_uint64, c_uint32, c_uint32, c_uint64, c_void_p]
        L.sr_downcast_f32_fp4.restype = c_int
        L.sr_accumulate_bf16.argtypes = [c_void_p, c_void_p, c_int, c_uint64, c_float, c_uint32, c_uint64, c_uint32,
                                         c_uint32, c_uint64, c_void_p]
        L.sr_accumulate_bf16.restype = c_int
        L.sr_adamw_step.argtypes = [c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_uint64, POINTER(HParams),
                                    c_uint64, c_uint32, c_uint32, c_uint64, c_void_p]
        L.sr_adamw_step.restype = c_int
        L.sr_master_adamw_step.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_uint64,
                                           POINTER(HParams), c_uint32, c_void_p]
        L.sr_master_adamw_step.restype = c_int
        L.sr_adamw_step_host_staging_bytes.argtypes = [c_int, c_uint64]
        L.sr_adamw_step_host_staging_bytes.restype = c_size_t
        L.sr_adamw_step_host.argtypes = [c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_uint64, POINTER(HParams),
                                         c_uint64, c_uint32, c_uint32, c_uint64, c_void_p, c_size_t, c_uint64, c_void_p]
        L.sr_adamw_step_host.restype = c_int
        L.sr_mt_plan_create.argtypes = [POINTER(c_void_p), c_uint32, POINTER(c_void_p), POINTER(c_void_p),
                                        POINTER(c_void_p), POINTER(c_void_p), POINTER(c_uint64), c_int, c_void_p]
        L.sr_mt_plan_create.restype = c_int
        L.sr_adamw_multi_tensor.argtypes = [c_void_p, POINTER(HParams), c_uint64, c_uint32, c_uint32, c_void_p]
        L.sr_adamw_multi_tensor.restype = c_int
        L.sr_mt_plan_destroy.argtypes = [c_void_p]
        L.sr_mt_plan_destroy.restype = c_int
        L.sr_mt_plan_total_elements.argtypes = [c_void_p]
        L.sr_mt_plan_total_elements.restype = c_uint64
        L.grad_sqnorm_multi_tensor_workspace_bytes.argtypes = [c_void_p]
        L.grad_sqnorm_multi_tensor_workspace_bytes.restype = c_size_t
        L.grad_sqnorm_multi_tensor.argtypes = [c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.grad_sqnorm_multi_tensor.restype = c_int
        L.grad_sqnorm_workspace_bytes.argtypes = [c_uint64]
        L.grad_sqnorm_workspace_bytes.restype = c_size_t
        L.grad_sqnorm.argtypes = [c_void_p, c_int, c_uint64, c_void_p, c_void_p, c_size_t, c_void_p]
        L.grad_sqnorm.restype = c_int
        L.grad_sqnorm_static.argtypes = [c_void_p, c_int, c_uint64, c_void_p, c_void_p]
        L.grad_sqnorm_static.restype = c_int
        L.grad_sqnorm_static_max_elements.restype = c_uint64
        L.sr_clip_scale.argtypes = [c_void_p, c_float, c_float, c_void_p, c_void_p]
        L.sr_clip_scale.restype = c_int
        L.sr_adamw_step_launch_count.argtypes = [c_uint64, c_uint64]
        L.sr_adamw_step_launch_count.restype = c_uint32
        L.sr_selftest_in_range_arithmetic.argtypes = [c_uint64, c_uint64, c_void_p, c_void_p]
        L.sr_selftest_in_range_arithmetic.restype = c_int
        L.sr_status_string.argtypes = [c_int]
        L.sr_status_string.restype = c_char_p
        L.sr_last_cuda_error.restype = c_int
        L.sr_abi_version.restype = c_uint32
        _lib = L
    return _lib


def _want(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def _stream(stream: Optional[torch.cuda.Stream]) -> c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return c_void_p(s.cuda_stream)


def _g_dtype(g: torch.Tensor) -> int:
    if g.dtype == torch.bfloat16:
        return SR_DT_BF16
    if g.dtype == torch.float32:
        return SR_DT_F32
    raise TypeError("gradient must be bfloat16 or float32")


def _check(status: int, where: str) -> None:
    if status != SR_OK:
        raise SrError(status, where)


def sr_downcast_f32_bf16(src: torch.Tensor, dst: torch.Tensor, seed: int, step: int = 0, tensor_id: int = 0,
                         elem_offset: int = 0, stream=None) -> None:
    _want(src, torch.float32, "src"), _want(dst, torch.bfloat16, "dst")
    if src.numel() != dst.numel():
        raise ValueError("size mismatch")
    with torch.cuda.device(src.device):
        _check(lib().sr_downcast_f32_bf16(src.data_ptr(), dst.data_ptr(), src.numel(), seed, step, tensor_id,
                                          elem_offset, _stream(stream)), "sr_downcast_f32_bf16")


SR_FP8_E4M3, SR_FP8_E5M2 = 0, 1


def sr_downcast_f32_fp8(src: torch.Tensor, dst: torch.Tensor, seed: int, step: int = 0, tensor_id: int = 0,
                        elem_offset: int = 0, stream=None) -> None:
    """dst: torch.float8_e4m3fn, torch.float8_e5m2 (the format follows the dtype) or uint8 (E4M3)."""
    _want(src, torch.float32, "src")
    if not dst.is_cuda or not dst.is_contiguous() or dst.element_size() != 1:
        raise TypeError("dst: expected a contiguous CUDA tensor of an 8-bit type")
    fmt = SR_FP8_E5M2 if dst.dtype == torch.float8_e5m2 else SR_FP8_E4M3
    if src.numel() != dst.numel():
        raise ValueError("size mismatch")
    with torch.cuda.device(src.device):
        _check(lib().sr_downcast_f32_fp8(src.data_ptr(), dst.data_ptr(), src.numel(), fmt, seed, step, tensor_id,
                                         elem_offset, _stream(stream)), "sr_downcast_f32_fp8")


def sr_downcast_f32_fp4(src: torch.Tensor, dst: torch.Tensor, seed: int, step: int = 0, tensor_id: int = 0,
                        elem_offset: int = 0, stream=None) -> None:
    """dst: (n + 1) // 2 bytes (uint8), two E2M1 codes per byte, the even element in the low half."""
    _want(src, torch.float32, "src"), _want(dst, torch.uint8, "dst")
    if dst.numel() != (src.numel() + 1) // 2:
        raise ValueError("size mismatch")
    with torch.cuda.device(src.device):
        _check(lib().sr_downcast_f32_fp4(src.data_ptr(), dst.data_ptr(), src.numel(), seed, step, tensor_id, elem_offset,
                                         _stream(stream)), "sr_downcast_f32_fp4")


def sr_accumulate_bf16(acc: torch.Tensor, g: torch.Tensor, scale: float = 1.0, seed: int = 0, step: int = 0,
                       tensor_id: int = 0, elem_offset: int = 0, stochastic: bool = True, stream=None) -> None:
    """acc (BF16, in place) <- rounding(acc + scale * g); g is BF16 or FP32."""
    _want(acc, torch.bfloat16, "acc"), _want(g, g.dtype, "g")
    if g.numel() != acc.numel():
        raise ValueError("size mismatch")
    with torch.cuda.device(acc.device):
        _check(lib().sr_accumulate_bf16(acc.data_ptr(), g.data_ptr(), _g_dtype(g), acc.numel(), scale,
                                        SR_FLAG_SR_P if stochastic else 0, seed, step, tensor_id, elem_offset,
                                        _stream(stream)), "sr_accumulate_bf16")


def sr_adamw_step(p: torch.Tensor, g: torch.Tensor, m: torch.Tensor, v: torch.Tensor, hp: HParams, seed: int,
                  step: int, tensor_id: int = 0, elem_offset: int = 0, stream=None) -> None:
    _want(p, torch.bfloat16, "p"), _want(m, torch.bfloat16, "m"), _want(v, torch.bfloat16, "v")
    _want(g, g.dtype, "g")
    n = p.numel()
    if not (g.numel() == m.numel() == v.numel() == n):
        raise ValueError("size mismatch")
    with torch.cuda.device(p.device):
        _check(lib().sr_adamw_step(p.data_ptr(), g.data_ptr(), _g_dtype(g), m.data_ptr(), v.data_ptr(), n,
                                   ctypes.byref(hp), seed, step, tensor_id, elem_offset, _stream(stream)),
               "sr_adamw_step")


def sr_master_adamw_step(p: torch.Tensor, p_bf16: torch.Tensor, g: torch.Tensor, m: torch.Tensor, v: torch.Tensor,
                         hp: HParams, step: int, stream=None) -> None:
    """FP32 master weights / moments (in place) with a nearest-rounded BF16 copy of x: the paper's
    mixed-precision comparison recipe."""
    _want(p, torch.float32, "p"), _want(m, torch.float32, "m"), _want(v, torch.float32, "v")
    _want(p_bf16, torch.bfloat16, "p_bf16"), _want(g, g.dtype, "g")
    n = p.numel()
    if not (g.numel() == m.numel() == v.numel() == p_bf16.numel() == n):
        raise ValueError("size mismatch")
    with torch.cuda.device(p.device):
        _check(lib().sr_master_adamw_step(p.data_ptr(), p_bf16.data_ptr(), g.data_ptr(), _g_dtype(g), m.data_ptr(),
                                          v.data_ptr(), n, ctypes.byref(hp), step, _stream(stream)),
               "sr_master_adamw_step")


def sr_adamw_step_host_staging_bytes(g_dtype: torch.dtype, chunk_elems: int) -> int:
    return int(lib().sr_adamw_step_host_staging_bytes(SR_DT_F32 if g_dtype == torch.float32 else SR_DT_BF16, chunk_elems))


def sr_adamw_step_host(p: torch.Tensor, g: torch.Tensor, m: torch.Tensor, v: torch.Tensor, hp: HParams, seed: int,
                       step: int, staging: torch.Tensor, chunk_elems: int, tensor_id: int = 0, elem_offset: int = 0,
                       stream=None) -> None:
    """p, g, m, v: HOST tensors (pinned for asynchronous copies); staging: CUDA scratch tensor.
    The host tensors must stay alive and untouched until the stream has been synchronised."""
    for t, name in ((p, "p"), (m, "m"), (v, "v")):
        if t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise TypeError(f"{name}: expected a contiguous host bfloat16 tensor")
    if g.is_cuda or not g.is_contiguous():
        raise TypeError("g: expected a contiguous host tensor")
    if not staging.is_cuda:
        raise TypeError("staging: expected a CUDA tensor")
    n = p.numel()
    if not (g.numel() == m.numel() == v.numel() == n):
        raise ValueError("size mismatch")
    with torch.cuda.device(staging.device):
        _check(lib().sr_adamw_step_host(p.data_ptr(), g.data_ptr(), _g_dtype(g), m.data_ptr(), v.data_ptr(), n,
                                        ctypes.byref(hp), seed, step, tensor_id, elem_offset, staging.data_ptr(),
                                        staging.numel() * staging.element_size(), chunk_elems, _stream(stream)),
               "sr_adamw_step_host")


class MtPlan:
    """Owns an ``sr_mt_plan`` and keeps the tensors it names alive."""

    def __init__(self, p: Sequence[torch.Tensor], g: Sequence[torch.Tensor], m: Sequence[torch.Tensor],
                 v: Sequence[torch.Tensor], stream=None):
        k = len(p)
        if not (len(g) == len(m) == len(v) == k):
            raise ValueError("list length mismatch")
        g_dt = _g_dtype(g[0]) if k else SR_DT_BF16
        for i in range(k):
            _want(p[i], torch.bfloat16, "p"), _want(m[i], torch.bfloat16, "m"), _want(v[i], torch.bfloat16, "v")
            if _g_dtype(_want(g[i], g[i].dtype, "g")) != g_dt:
                raise TypeError("all gradients of a list share one dtype")
            if not (g[i].numel() == m[i].numel() == v[i].numel() == p[i].numel()):
                raise ValueError("size mismatch")
        self._keep = (list(p), list(g), list(m), list(v))
        arr = lambda ts: (c_void_p * k)(*[t.data_ptr() for t in ts])
        numel = (c_uint64 * k)(*[t.numel() for t in p])
        self._handle = c_void_p()
        self.device = p[0].device if k else torch.device("cuda", torch.cuda.current_device())
        with torch.cuda.device(self.device):
            _check(lib().sr_mt_plan_create(ctypes.byref(self._handle), k, arr(p), arr(g), arr(m), arr(v), numel,
                                           g_dt, _stream(stream)), "sr_mt_plan_create")

    @property
    def total_elements(self) -> int:
        return int(lib().sr_mt_plan_total_elements(self._handle))

    def destroy(self) -> None:
        if self._handle:
            h, self._handle = self._handle, c_void_p()
            _check(lib().sr_mt_plan_destroy(h), "sr_mt_plan_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def sr_mt_plan_create(p, g, m, v, stream=None) -> MtPlan:
    return MtPlan(p, g, m, v, stream)


def sr_adamw_multi_tensor(plan: MtPlan, hp: HParams, seed: int, step: int, tensor_id_base: int = 0, stream=None) -> None:
    with torch.cuda.device(plan.device):
        _check(lib().sr_adamw_multi_tensor(plan._handle, ctypes.byref(hp), seed, step, tensor_id_base,
                                           _stream(stream)), "sr_adamw_multi_tensor")


def sr_mt_plan_destroy(plan: MtPlan) -> None:
    plan.destroy()


def grad_sqnorm_workspace_bytes(n: int) -> int:
    return int(lib().grad_sqnorm_workspace_bytes(n))


def grad_sqnorm(g: torch.Tensor, out: torch.Tensor, workspace: Optional[torch.Tensor], stream=None) -> None:
    """out: one float64 on the device.  workspace: any CUDA tensor of at least
    grad_sqnorm_workspace_bytes(g.numel()) bytes (or None when that is 0)."""
    _want(g, g.dtype, "g"), _want(out, torch.float64, "out")
    ws_ptr, ws_bytes = (workspace.data_ptr(), workspace.numel() * workspace.element_size()) if workspace is not None else (None, 0)
    with torch.cuda.device(g.device):
        _check(lib().grad_sqnorm(g.data_ptr(), _g_dtype(g), g.numel(), out.data_ptr(), ws_ptr, ws_bytes,
                                 _stream(stream)), "grad_sqnorm")


def grad_sqnorm_multi_tensor_workspace_bytes(plan: MtPlan) -> int:
    return int(lib().grad_sqnorm_multi_tensor_workspace_bytes(plan._handle))


def grad_sqnorm_multi_tensor(plan: MtPlan, out: torch.Tensor, workspace: Optional[torch.Tensor], stream=None) -> None:
    """Sum of squares over all gradients of the plan's list; out: one float64 on the device."""
    _want(out, torch.float64, "out")
    ws_ptr, ws_bytes = (workspace.data_ptr(), workspace.numel() * workspace.element_size()) if workspace is not None else (None, 0)
    with torch.cuda.device(plan.device):
        _check(lib().grad_sqnorm_multi_tensor(plan._handle, out.data_ptr(), ws_ptr, ws_bytes, _stream(stream)),
               "grad_sqnorm_multi_tensor")


def grad_sqnorm_static_max_elements() -> int:
    return int(lib().grad_sqnorm_static_max_elements())


def grad_sqnorm_static(g: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """grad_sqnorm without a workspace: the block sums go to a fixed array inside the library, so the
    call allocates nothing.  For callers that may not allocate device memory; all such calls on one
    GPU share that array, so do not let two of them overlap.  g.numel() is limited to
    grad_sqnorm_static_max_elements()."""
    _want(g, g.dtype, "g"), _want(out, torch.float64, "out")
    with torch.cuda.device(g.device):
        _check(lib().grad_sqnorm_static(g.data_ptr(), _g_dtype(g), g.numel(), out.data_ptr(), _stream(stream)),
               "grad_sqnorm_static")


def sr_clip_scale(sqnorm: torch.Tensor, accum_scale: float, max_norm: float, gscale_out: torch.Tensor, stream=None) -> None:
    _want(sqnorm, torch.float64, "sqnorm"), _want(gscale_out, torch.float32, "gscale_out")
    with torch.cuda.device(sqnorm.device):
        _check(lib().sr_clip_scale(sqnorm.data_ptr(), accum_scale, max_norm, gscale_out.data_ptr(), _stream(stream)),
               "sr_clip_scale")


def sr_adamw_step_launch_count(n: int, elem_offset: int = 0) -> int:
    """Kernel launches that one sr_adamw_step call of n elements at elem_offset enqueues."""
    return int(lib().sr_adamw_step_launch_count(n, elem_offset))


def sr_selftest_in_range_arithmetic(seed: int, sets: int, mismatches: torch.Tensor, stream=None) -> None:
    """Compare the step kernels' branch-free square root and division with the IEEE instructions on `sets` seeded
    operand sets; mismatches (two int64 on the device) receives the counts (square roots, divisions)."""
    _want(mismatches, torch.int64, "mismatches")
    if mismatches.numel() < 2:
        raise ValueError("mismatches needs two elements")
    with torch.cuda.device(mismatches.device):
        _check(lib().sr_selftest_in_range_arithmetic(seed, sets, mismatches.data_ptr(), _stream(stream)),
               "sr_selftest_in_range_arithmetic")


def sr_abi_version() -> int:
    return int(lib().sr_abi_version())
