"""CPU oracle for FPROP direct convolution — TEST INFRASTRUCTURE ONLY.

A plain fp64-accumulating restatement of the paper's definition (Section 2) in
C (``conv_oracle.c``), loaded through ctypes.  Only the tests, the smoke check
and the benchmark's CPU-baseline / reference legs may import this package; the
product path never does, and this package imports nothing from the product.

Pinned by ``tests/test_oracle_pins.py`` (hand-worked examples, brute-force
loops, an im2col formulation, library convolution, closed forms, invariants).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


class ConvDesc(ctypes.Structure):
    """Section 2's symbols, in the boundary's field order."""

    _fields_ = [
        ("Nb", ctypes.c_int32), ("Wi", ctypes.c_int32), ("Hi", ctypes.c_int32),
        ("Nc", ctypes.c_int32), ("No", ctypes.c_int32), ("Sk", ctypes.c_int32),
        ("stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("alpha", ctypes.c_float),
    ]


def build(force: bool = False) -> str:
    """Compile ``conv_oracle.c`` into ``liboracle.so`` beside it (gcc, OpenMP)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.POINTER
        lib.oracle_conv_out_dims.restype = ctypes.c_int
        lib.oracle_conv_out_dims.argtypes = [P(ConvDesc), P(ctypes.c_int32), P(ctypes.c_int32)]
        lib.oracle_conv_flops.restype = ctypes.c_uint64
        lib.oracle_conv_flops.argtypes = [P(ConvDesc)]
        lib.oracle_conv_fprop.restype = ctypes.c_int
        lib.oracle_conv_fprop.argtypes = [P(ConvDesc), ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_int32]
        lib.oracle_conv_fprop_rows.restype = ctypes.c_int
        lib.oracle_conv_fprop_rows.argtypes = [P(ConvDesc), ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                               ctypes.c_int32]
        lib.oracle_conv_fprop_point.restype = ctypes.c_double
        lib.oracle_conv_fprop_point.argtypes = [P(ConvDesc), ctypes.c_void_p, ctypes.c_void_p,
                                                ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                                ctypes.c_int32, P(ctypes.c_double)]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha) -> ConvDesc:
    return ConvDesc(int(Nb), int(Wi), int(Hi), int(Nc), int(No), int(Sk), int(stride),
                    int(pad), float(alpha))


def out_dims(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha=1.0):
    """(Ho, Wo) = floor((in + 2 pad - Sk)/stride) + 1 per axis; ValueError if empty."""
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    if _load().oracle_conv_out_dims(ctypes.byref(d), ctypes.byref(ho), ctypes.byref(wo)):
        raise ValueError("invalid convolution descriptor")
    return ho.value, wo.value


def flops(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha=1.0) -> int:
    """The paper's complexity formula C (Section 2)."""
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    return int(_load().oracle_conv_flops(ctypes.byref(d)))


def _check(a, shape, name):
    a = np.ascontiguousarray(a, dtype=np.float32)
    if a.shape != tuple(shape):
        raise ValueError("%s has shape %s, expected %s" % (name, a.shape, tuple(shape)))
    return a


def conv_fprop(inp, filt, *, stride=1, pad=0, alpha=1.0, nthreads=0, rows=None):
    """out[No,Ho,Wo,Nb] from in[Nc,Hi,Wi,Nb] and filt[Nc,Sk,Sk,No] (fp32 arrays).

    ``rows=(y0, y1)`` computes only output rows y0 <= y < y1 (other rows are
    left at zero) — used to time a bounded sample of a large workload.
    """
    inp = np.ascontiguousarray(inp, dtype=np.float32)
    filt = np.ascontiguousarray(filt, dtype=np.float32)
    Nc, Hi, Wi, Nb = inp.shape
    Nc2, Sk, Sk2, No = filt.shape
    if Nc2 != Nc or Sk2 != Sk:
        raise ValueError("filter bank does not match the maps")
    Ho, Wo = out_dims(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    out = np.zeros((No, Ho, Wo, Nb), dtype=np.float32)
    y0, y1 = (0, Ho) if rows is None else rows
    rc = _load().oracle_conv_fprop_rows(ctypes.byref(d), inp.ctypes.data, filt.ctypes.data,
                                        out.ctypes.data, int(y0), int(y1), int(nthreads))
    if rc:
        raise RuntimeError("oracle_conv_fprop_rows failed (%d)" % rc)
    return out


def conv_fprop_point(inp, filt, o, y, x, n, *, stride=1, pad=0, alpha=1.0):
    """(value, abs_sum) of one output element in fp64 (value is not rounded to fp32)."""
    inp = np.ascontiguousarray(inp, dtype=np.float32)
    filt = np.ascontiguousarray(filt, dtype=np.float32)
    Nc, Hi, Wi, Nb = inp.shape
    _, Sk, _, No = filt.shape
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    a = ctypes.c_double()
    v = _load().oracle_conv_fprop_point(ctypes.byref(d), inp.ctypes.data, filt.ctypes.data,
                                        int(o), int(y), int(x), int(n), ctypes.byref(a))
    return float(v), float(a.value)


def num_threads() -> int:
    return int(_load().oracle_num_threads())
