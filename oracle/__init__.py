"""ctypes access to the CPU oracle (``sradamw_oracle.cpp``).

Test infrastructure only: the CUDA library and its Python binding never import this package.
Arrays are numpy arrays in host memory; BF16 values travel as ``uint16`` bit patterns.
"""

from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_uint16, c_uint32, c_uint64, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sradamw_oracle.cpp")
_LIB = os.path.join(_HERE, "libsradamw_oracle.so")

SR_P, SR_M, SR_V = 1, 2, 4
EPS_INSIDE = 8
SR_ALL = SR_P | SR_M | SR_V


class HParams(ctypes.Structure):
    _fields_ = [
        ("lr", c_float),
        ("beta1", c_float),
        ("beta2", c_float),
        ("eps", c_float),
        ("weight_decay", c_float),
        ("flags", c_uint32),
    ]


class Scalars(ctypes.Structure):
    _fields_ = [
        ("beta1", c_float),
        ("beta2", c_float),
        ("one_minus_beta1", c_float),
        ("one_minus_beta2", c_float),
        ("step_size", c_float),
        ("rsqrt_bc2", c_float),
        ("eps", c_float),
        ("lr_wd", c_float),
        ("inv_bc2", c_float),
        ("eps_inside", c_uint32),
    ]


class Trace(ctypes.Structure):
    _fields_ = [(name, c_float) for name in
                ("g", "a", "m_new", "b1", "b2", "v_new", "s", "den", "u", "w", "q", "x_new")]


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no contraction, baseline x86-64 so the same
    binary runs on any host).  Returns the path of the shared library."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-Wall", "-Wextra", _SRC, "-o", _LIB]
    subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_num_threads.restype = c_int
        L.oracle_philox4x32_10.argtypes = [POINTER(c_uint32), POINTER(c_uint32), POINTER(c_uint32)]
        L.oracle_noise.argtypes = [c_uint64, c_uint32, c_uint32, c_uint64, POINTER(c_uint32)]
        L.oracle_sr_bf16_bits.argtypes = [c_uint32, c_uint32]
        L.oracle_sr_bf16_bits.restype = c_uint16
        L.oracle_rne_bf16_bits.argtypes = [c_uint32]
        L.oracle_rne_bf16_bits.restype = c_uint16
        L.oracle_adamw_scalars.argtypes = [POINTER(HParams), c_uint32, POINTER(Scalars)]
        L.oracle_adamw_scalars.restype = c_int
        L.oracle_adamw_element.argtypes = [c_float, c_float, c_float, c_float, c_float,
                                           POINTER(Scalars), POINTER(Trace)]
        L.oracle_adamw_step.argtypes = [c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_uint64,
                                        POINTER(HParams), c_float, c_uint64, c_uint32, c_uint32, c_uint64]
        L.oracle_adamw_step.restype = c_int
        L.oracle_master_adamw_step.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_uint64,
                                               POINTER(HParams), c_float, c_uint32]
        L.oracle_master_adamw_step.restype = c_int
        L.oracle_sr_fp8_bits.argtypes = [c_uint32, c_uint32, c_int]
        L.oracle_sr_fp8_bits.restype = ctypes.c_uint8
        L.oracle_noise32.argtypes = [c_uint64, c_uint32, c_uint32, c_uint64]
        L.oracle_noise32.restype = c_uint32
        L.oracle_sr_downcast_fp8.argtypes = [c_void_p, c_void_p, c_uint64, c_int, c_uint64, c_uint32, c_uint32, c_uint64]
        L.oracle_sr_downcast.argtypes = [c_void_p, c_void_p, c_uint64, c_uint64, c_uint32, c_uint32, c_uint64]
        L.oracle_sr_fp4_bits.argtypes = [c_uint32, c_uint32]
        L.oracle_sr_fp4_bits.restype = ctypes.c_uint8
        L.oracle_sr_downcast_fp4.argtypes = [c_void_p, c_void_p, c_uint64, c_uint64, c_uint32, c_uint32, c_uint64]
        L.oracle_noise_slot.argtypes = [c_uint64, c_uint32, c_uint32, c_uint64, c_uint32]
        L.oracle_noise_slot.restype = c_uint32
        L.oracle_accumulate_element.argtypes = [ctypes.c_uint16, c_float, c_float, c_uint32, c_int]
        L.oracle_accumulate_element.restype = ctypes.c_uint16
        L.oracle_sr_accumulate.argtypes = [c_void_p, c_void_p, c_int, c_uint64, c_float, c_int, c_uint64, c_uint32,
                                           c_uint32, c_uint64]
        L.oracle_sqnorm.argtypes = [c_void_p, c_int, c_uint64]
        L.oracle_sqnorm.restype = c_double
        L.oracle_tree_sum.argtypes = [c_void_p, c_uint64]
        L.oracle_tree_sum.restype = c_double
        L.oracle_clip_scale.argtypes = [c_double, c_float, c_float]
        L.oracle_clip_scale.restype = c_float
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _check(a: np.ndarray, dtype) -> np.ndarray:
    if a.dtype != np.dtype(dtype) or not a.flags["C_CONTIGUOUS"]:
        raise TypeError(f"expected contiguous {np.dtype(dtype)} array, got {a.dtype}")
    return a


def _ptr(a: np.ndarray) -> c_void_p:
    return c_void_p(a.ctypes.data)


def philox4x32_10(ctr, key):
    c = (c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    out = (c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, out)
    return tuple(int(x) for x in out)


def noise(seed: int, step: int, tensor_id: int, index: int):
    out = (c_uint32 * 3)()
    lib().oracle_noise(seed, step, tensor_id, index, out)
    return tuple(int(x) for x in out)


def sr_bf16_bits(fbits: int, r16: int) -> int:
    return int(lib().oracle_sr_bf16_bits(fbits & 0xFFFFFFFF, r16))


def rne_bf16_bits(fbits: int) -> int:
    return int(lib().oracle_rne_bf16_bits(fbits & 0xFFFFFFFF))


def hparams(lr, beta1, beta2, eps, weight_decay, flags=SR_ALL) -> HParams:
    return HParams(lr, beta1, beta2, eps, weight_decay, flags)


def adamw_scalars(hp: HParams, step: int) -> Scalars:
    sc = Scalars()
    if lib().oracle_adamw_scalars(ctypes.byref(hp), step, ctypes.byref(sc)) != 0:
        raise ValueError("AdamW is not defined for step 0")
    return sc


def adamw_element(x, g, m, v, gscale, sc: Scalars) -> Trace:
    t = Trace()
    lib().oracle_adamw_element(x, g, m, v, gscale, ctypes.byref(sc), ctypes.byref(t))
    return t


def adamw_step(p, g, m, v, hp: HParams, seed, step, tensor_id=0, elem_offset=0, gscale=1.0):
    """In place on uint16 arrays p, m, v; g is uint16 (BF16 bits) or float32."""
    _check(p, np.uint16), _check(m, np.uint16), _check(v, np.uint16)
    if g.dtype == np.float32:
        g_is_f32 = 1
    else:
        _check(g, np.uint16)
        g_is_f32 = 0
    n = p.size
    if not (g.size == m.size == v.size == n):
        raise ValueError("size mismatch")
    rc = lib().oracle_adamw_step(_ptr(p), _ptr(g), g_is_f32, _ptr(m), _ptr(v), n, ctypes.byref(hp),
                                 gscale, seed, step, tensor_id, elem_offset)
    if rc != 0:
        raise ValueError("AdamW is not defined for step 0")


def master_adamw_step(p, g, m, v, hp: HParams, step, gscale=1.0):
    """FP32 master recipe, in place on float32 arrays p, m, v; g is uint16 (BF16 bits) or float32.
    Returns the BF16 copy of the updated parameters (uint16 bit patterns)."""
    _check(p, np.float32), _check(m, np.float32), _check(v, np.float32)
    g_is_f32 = 1 if g.dtype == np.float32 else 0
    if not g_is_f32:
        _check(g, np.uint16)
    n = p.size
    if not (g.size == m.size == v.size == n):
        raise ValueError("size mismatch")
    p16 = np.empty(p.shape, dtype=np.uint16)
    rc = lib().oracle_master_adamw_step(_ptr(p), _ptr(p16), _ptr(g), g_is_f32, _ptr(m), _ptr(v), n, ctypes.byref(hp),
                                        gscale, step)
    if rc != 0:
        raise ValueError("AdamW is not defined for step 0")
    return p16


def sr_downcast(src, seed, step=0, tensor_id=0, elem_offset=0):
    _check(src, np.float32)
    dst = np.empty(src.shape, dtype=np.uint16)
    lib().oracle_sr_downcast(_ptr(src), _ptr(dst), src.size, seed, step, tensor_id, elem_offset)
    return dst


def sr_fp8_bits(fbits: int, r32: int, e5m2: bool) -> int:
    return int(lib().oracle_sr_fp8_bits(fbits & 0xFFFFFFFF, r32 & 0xFFFFFFFF, 1 if e5m2 else 0))


def noise32(seed: int, step: int, tensor_id: int, index: int) -> int:
    return int(lib().oracle_noise32(seed, step, tensor_id, index))


def sr_downcast_fp8(src, e5m2: bool, seed, step=0, tensor_id=0, elem_offset=0):
    _check(src, np.float32)
    dst = np.empty(src.shape, dtype=np.uint8)
    lib().oracle_sr_downcast_fp8(_ptr(src), _ptr(dst), src.size, 1 if e5m2 else 0, seed, step, tensor_id, elem_offset)
    return dst


def sr_fp4_bits(fbits: int, r32: int) -> int:
    """Code (sign bit 3, magnitude bits 0..2) of Q_SR on the E2M1 grid for one FP32 pattern and one noise word."""
    return int(lib().oracle_sr_fp4_bits(fbits & 0xFFFFFFFF, r32 & 0xFFFFFFFF))


def sr_downcast_fp4(src, seed, step=0, tensor_id=0, elem_offset=0):
    """Packed E2M1 codes, two per byte (even element in the low half)."""
    _check(src, np.float32)
    dst = np.empty((src.size + 1) // 2, dtype=np.uint8)
    lib().oracle_sr_downcast_fp4(_ptr(src), _ptr(dst), src.size, seed, step, tensor_id, elem_offset)
    return dst


def noise_slot(seed: int, step: int, tensor_id: int, index: int, slot: int) -> int:
    """16-bit noise of rounding slot 0..3 of one element."""
    return int(lib().oracle_noise_slot(seed, step, tensor_id, index, slot))


def accumulate_element(acc_bits: int, g: float, scale: float, r16: int, stochastic: bool = True) -> int:
    return int(lib().oracle_accumulate_element(acc_bits & 0xFFFF, g, scale, r16 & 0xFFFF, 1 if stochastic else 0))


def sr_accumulate(acc, g, scale, seed, step, tensor_id=0, elem_offset=0, stochastic=True):
    """In place: acc (BF16 bit patterns, uint16) <- rounding(acc + scale * g); g is uint16 (BF16) or float32."""
    _check(acc, np.uint16)
    if g.dtype == np.float32:
        _check(g, np.float32)
        is32 = 1
    else:
        _check(g, np.uint16)
        is32 = 0
    assert g.size == acc.size
    lib().oracle_sr_accumulate(_ptr(acc), _ptr(g), is32, acc.size, scale, 1 if stochastic else 0, seed, step, tensor_id,
                               elem_offset)
    return acc


def sqnorm(g) -> float:
    if g.dtype == np.float32:
        return float(lib().oracle_sqnorm(_ptr(_check(g, np.float32)), 1, g.size))
    return float(lib().oracle_sqnorm(_ptr(_check(g, np.uint16)), 0, g.size))


def sqnorm_list(grads) -> float:
    """Sum of squares over a list of gradient arrays: one block sum per chunk of 8192 consecutive entries of
    each array (arrays in list order, the block rule applied inside the chunk), then the array of block sums
    reduced by the tree.  Composed from the two routines above."""
    partials = []
    for g in grads:
        flat = np.ascontiguousarray(g).reshape(-1)
        for start in range(0, flat.size, 8192):
            partials.append(sqnorm(np.ascontiguousarray(flat[start:start + 8192])))
    if not partials:
        return 0.0
    if len(partials) == 1:
        return partials[0]
    return tree_sum(np.array(partials, dtype=np.float64))


def tree_sum(terms) -> float:
    _check(terms, np.float64)
    return float(lib().oracle_tree_sum(_ptr(terms), terms.size))


def clip_scale(sqnorm_value: float, accum_scale: float, max_norm: float) -> float:
    return float(lib().oracle_clip_scale(sqnorm_value, accum_scale, max_norm))
