"""ctypes front end of the CPU oracle (``sifar_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's
CPU-baseline leg call this; the GPU library never does, and this module never
imports the GPU package.  bf16 tensors travel as ``numpy.uint16`` bit patterns,
fp32 tensors as ``numpy.float32``.

The reduction follows Section 3.1 ("Oneshot", phase 2) of the paper: element-wise
sum over ranks in rank order, here fixed to binary32 accumulation and a single
round-to-nearest-even to the output type.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sifar_oracle.c")
_LIB = os.path.join(_HERE, "libsifar_oracle.so")

BF16, F32 = 0, 1
KIND_GAUSS, KIND_INT, KIND_UNIFORM = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-std=c11", "-O1", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
             "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class Workload(ctypes.Structure):
    """Mirror of ``oracle_workload`` (see the C file for the update rules)."""
    _fields_ = [("kind", ctypes.c_int32), ("seed", ctypes.c_uint32),
                ("scale", ctypes.c_float), ("sigma", ctypes.c_float),
                ("outlier_mod", ctypes.c_uint32), ("delay_max_ns", ctypes.c_uint32)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32, i32, f32 = ctypes.c_uint32, ctypes.c_int32, ctypes.c_float
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        L.oracle_bf16_to_f32.restype = f32
        L.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        L.oracle_f32_to_bf16.restype = ctypes.c_uint16
        L.oracle_f32_to_bf16.argtypes = [f32]
        L.oracle_f32_to_bf16_array.restype = None
        L.oracle_f32_to_bf16_array.argtypes = [vp, sz, vp]
        L.oracle_bf16_to_f32_array.restype = None
        L.oracle_bf16_to_f32_array.argtypes = [vp, sz, vp]
        for name in ("oracle_allreduce_bf16", "oracle_allreduce_f32"):
            getattr(L, name).restype = None
            getattr(L, name).argtypes = [vp, ctypes.c_int, sz, vp]
        L.oracle_gen_word.restype = u32
        L.oracle_gen_word.argtypes = [u32] * 6
        for name in ("oracle_gen_uniform", "oracle_gen_gauss"):
            getattr(L, name).restype = f32
            getattr(L, name).argtypes = [u32] * 4
        L.oracle_gen_int129.restype = i32
        L.oracle_gen_int129.argtypes = [u32] * 4
        L.oracle_gen_is_outlier.restype = ctypes.c_int
        L.oracle_gen_is_outlier.argtypes = [u32] * 4
        L.oracle_gen_delay_ns.restype = u32
        L.oracle_gen_delay_ns.argtypes = [u32] * 4
        wp = ctypes.POINTER(Workload)
        L.oracle_workload_first_bf16.restype = None
        L.oracle_workload_first_bf16.argtypes = [wp, ctypes.c_int, sz, vp]
        L.oracle_workload_first_f32.restype = None
        L.oracle_workload_first_f32.argtypes = [wp, ctypes.c_int, sz, vp]
        L.oracle_workload_next_bf16.restype = None
        L.oracle_workload_next_bf16.argtypes = [wp, ctypes.c_int, u32, sz, vp, vp]
        L.oracle_workload_next_f32.restype = None
        L.oracle_workload_next_f32.argtypes = [wp, ctypes.c_int, u32, sz, vp, vp]
        L.oracle_chain.restype = None
        L.oracle_chain.argtypes = [wp, ctypes.c_int, sz, ctypes.c_int, u32, ctypes.c_int, vp, vp, vp]
        _lib = L
    return _lib


def _np_dtype(dtype: int):
    return np.uint16 if dtype == BF16 else np.float32


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def f32_to_bf16(x) -> np.ndarray:
    """Element-wise RNE narrowing; accepts float32 values (bit patterns are preserved)."""
    L = lib()
    src = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(src.shape, dtype=np.uint16)
    L.oracle_f32_to_bf16_array(_ptr(src), src.size, _ptr(out))
    return out


def f32_bits_to_bf16(bits) -> np.ndarray:
    """Same, from binary32 bit patterns (NaN payloads and signed zeros reach C untouched)."""
    return f32_to_bf16(np.ascontiguousarray(bits, dtype=np.uint32).view(np.float32))


def bf16_to_f32(b) -> np.ndarray:
    """Exact widening through the C routine."""
    L = lib()
    src = np.ascontiguousarray(b, dtype=np.uint16)
    out = np.empty(src.shape, dtype=np.float32)
    L.oracle_bf16_to_f32_array(_ptr(src), src.size, _ptr(out))
    return out


def allreduce(xs, dtype: int) -> np.ndarray:
    """``xs``: sequence of P equally long 1-D arrays (uint16 bit patterns or float32)."""
    L = lib()
    nd = _np_dtype(dtype)
    arrs = [np.ascontiguousarray(x, dtype=nd) for x in xs]
    P, n = len(arrs), arrs[0].size
    assert P >= 1 and all(a.size == n for a in arrs)
    ptrs = (ctypes.c_void_p * P)(*[a.ctypes.data for a in arrs])
    out = np.empty(n, dtype=nd)
    fn = L.oracle_allreduce_bf16 if dtype == BF16 else L.oracle_allreduce_f32
    fn(ptrs, P, n, _ptr(out))
    return out


def workload_first(w: Workload, r: int, n: int, dtype: int) -> np.ndarray:
    L = lib()
    x = np.empty(n, dtype=_np_dtype(dtype))
    fn = L.oracle_workload_first_bf16 if dtype == BF16 else L.oracle_workload_first_f32
    fn(ctypes.byref(w), r, n, _ptr(x))
    return x


def workload_next(w: Workload, r: int, t: int, prev_out: np.ndarray, dtype: int) -> np.ndarray:
    L = lib()
    prev = np.ascontiguousarray(prev_out, dtype=_np_dtype(dtype))
    x = np.empty(prev.size, dtype=_np_dtype(dtype))
    fn = L.oracle_workload_next_bf16 if dtype == BF16 else L.oracle_workload_next_f32
    fn(ctypes.byref(w), r, t, prev.size, _ptr(prev), _ptr(x))
    return x


def chain(w: Workload, P: int, n: int, dtype: int, steps: int, t0: int = 1,
          out_prev: np.ndarray | None = None) -> np.ndarray:
    """Run ``steps`` dependent all-reduces from step ``t0``; returns ``[steps, n]``."""
    L = lib()
    nd = _np_dtype(dtype)
    outs = np.empty((steps, n), dtype=nd)
    scratch = np.empty(P * max(n, 1), dtype=nd)
    if t0 > 1:
        assert out_prev is not None
        prev = np.ascontiguousarray(out_prev, dtype=nd)
        pp = _ptr(prev)
    else:
        pp = ctypes.c_void_p(0)
    L.oracle_chain(ctypes.byref(w), P, n, dtype, t0, steps, pp, _ptr(outs), _ptr(scratch))
    return outs
