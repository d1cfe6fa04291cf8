"""CPU oracle for the direct convolution (FPROP and its two adjoints) — TEST INFRASTRUCTURE ONLY.

A plain fp64-accumulating restatement of the paper's definition (Section 2) in
C (``conv_oracle.c``) and of its gradients with respect to maps and filters
(``conv_bprop_oracle.c``), loaded through ctypes.  Only the tests, the smoke check
and the benchmark's CPU-baseline / reference legs may import this package; the
product path never does, and this package imports nothing from the product.

Pinned by ``tests/test_oracle_pins.py`` (hand-worked examples, brute-force
loops, an im2col formulation, library convolution, closed forms, invariants)
and ``tests/test_oracle_bprop_pins.py`` (adjoint identities against the pinned
FPROP, finite differences, brute-force loops, library autograd, closed forms).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_oracle.c")
_SRCS = [_SRC, os.path.join(_HERE, "conv_bprop_oracle.c")]
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
    """Compile the oracle's C files into ``liboracle.so`` beside them (gcc, OpenMP)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or any(os.path.getmtime(_LIB) < os.path.getmtime(p)
                                                  for p in _SRCS)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp] + _SRCS
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
        lib.oracle_conv2_out_dims.restype = ctypes.c_int
        lib.oracle_conv2_out_dims.argtypes = [P(ConvDesc2), P(ctypes.c_int32), P(ctypes.c_int32)]
        lib.oracle_conv2_fprop.restype = ctypes.c_int
        lib.oracle_conv2_fprop.argtypes = [P(ConvDesc2), ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_int32]
        for name in ("oracle_conv2_bprop_data", "oracle_conv2_bprop_filter"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [P(ConvDesc2), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                           ctypes.c_int32]
        for name in ("oracle_conv_bprop_data", "oracle_conv_bprop_filter"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [P(ConvDesc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                           ctypes.c_int32]
        for name in ("oracle_conv_bprop_data_point", "oracle_conv_bprop_filter_point"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_double
            fn.argtypes = [P(ConvDesc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                           ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, P(ctypes.c_double)]
        _lib = lib
    return _lib


class ConvDesc2(ctypes.Structure):
    """Per-axis filter size, stride and padding (w before h, as in the C struct)."""

    _fields_ = [(n, ctypes.c_int32) for n in ("Nb", "Wi", "Hi", "Nc", "No", "Skw", "Skh",
                                              "stride_w", "stride_h", "pad_w", "pad_h")] + \
               [("alpha", ctypes.c_float)]


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


def conv2_fprop(inp, filt, *, stride=(1, 1), pad=(0, 0), alpha=1.0, nthreads=0):
    """out[No,Ho,Wo,Nb] from in[Nc,Hi,Wi,Nb] and filt[Nc,Skh,Skw,No] with per-axis
    ``stride=(stride_h, stride_w)`` and ``pad=(pad_h, pad_w)``."""
    inp = np.ascontiguousarray(inp, dtype=np.float32)
    filt = np.ascontiguousarray(filt, dtype=np.float32)
    Nc, Hi, Wi, Nb = inp.shape
    Nc2, Skh, Skw, No = filt.shape
    if Nc2 != Nc:
        raise ValueError("filter bank does not match the maps")
    d = ConvDesc2(Nb, Wi, Hi, Nc, No, Skw, Skh, int(stride[1]), int(stride[0]), int(pad[1]),
                  int(pad[0]), float(alpha))
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    if _load().oracle_conv2_out_dims(ctypes.byref(d), ctypes.byref(ho), ctypes.byref(wo)):
        raise ValueError("invalid convolution descriptor")
    out = np.zeros((No, ho.value, wo.value, Nb), dtype=np.float32)
    rc = _load().oracle_conv2_fprop(ctypes.byref(d), inp.ctypes.data, filt.ctypes.data,
                                    out.ctypes.data, int(nthreads))
    if rc:
        raise RuntimeError("oracle_conv2_fprop failed (%d)" % rc)
    return out


def conv2_bprop_data(dout, filt, in_hw, *, stride=(1, 1), pad=(0, 0), alpha=1.0, nthreads=0):
    """din[Nc,Hi,Wi,Nb] for the per-axis operation; ``stride`` / ``pad`` are (h, w) pairs."""
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    filt = np.ascontiguousarray(filt, dtype=np.float32)
    No, Ho, Wo, Nb = dout.shape
    Nc, Skh, Skw, _ = filt.shape
    Hi, Wi = in_hw
    d = ConvDesc2(Nb, Wi, Hi, Nc, No, Skw, Skh, int(stride[1]), int(stride[0]), int(pad[1]),
                  int(pad[0]), float(alpha))
    din = np.zeros((Nc, Hi, Wi, Nb), dtype=np.float32)
    rc = _load().oracle_conv2_bprop_data(ctypes.byref(d), dout.ctypes.data, filt.ctypes.data,
                                         din.ctypes.data, int(nthreads))
    if rc:
        raise RuntimeError("oracle_conv2_bprop_data failed (%d)" % rc)
    return din


def conv2_bprop_filter(inp, dout, filt_hw, *, stride=(1, 1), pad=(0, 0), alpha=1.0, nthreads=0):
    """dfilt[Nc,Skh,Skw,No] for the per-axis operation; ``filt_hw`` = (Skh, Skw)."""
    inp = np.ascontiguousarray(inp, dtype=np.float32)
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    Nc, Hi, Wi, Nb = inp.shape
    No = dout.shape[0]
    Skh, Skw = filt_hw
    d = ConvDesc2(Nb, Wi, Hi, Nc, No, Skw, Skh, int(stride[1]), int(stride[0]), int(pad[1]),
                  int(pad[0]), float(alpha))
    dfilt = np.zeros((Nc, Skh, Skw, No), dtype=np.float32)
    rc = _load().oracle_conv2_bprop_filter(ctypes.byref(d), inp.ctypes.data, dout.ctypes.data,
                                           dfilt.ctypes.data, int(nthreads))
    if rc:
        raise RuntimeError("oracle_conv2_bprop_filter failed (%d)" % rc)
    return dfilt


def conv_bprop_data(dout, filt, in_hw, *, stride=1, pad=0, alpha=1.0, nthreads=0):
    """din[Nc,Hi,Wi,Nb] from dout[No,Ho,Wo,Nb] and filt[Nc,Sk,Sk,No]; ``in_hw`` = (Hi, Wi).

    The adjoint of FPROP with respect to the maps, alpha included.
    """
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    filt = np.ascontiguousarray(filt, dtype=np.float32)
    No, Ho, Wo, Nb = dout.shape
    Nc, Sk, Sk2, No2 = filt.shape
    Hi, Wi = in_hw
    if No2 != No or Sk2 != Sk or out_dims(Nb, Wi, Hi, Nc, No, Sk, stride, pad) != (Ho, Wo):
        raise ValueError("dout / filter bank / map size do not belong to one convolution")
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    din = np.zeros((Nc, Hi, Wi, Nb), dtype=np.float32)
    rc = _load().oracle_conv_bprop_data(ctypes.byref(d), dout.ctypes.data, filt.ctypes.data,
                                        din.ctypes.data, int(nthreads))
    if rc:
        raise RuntimeError("oracle_conv_bprop_data failed (%d)" % rc)
    return din


def conv_bprop_data_point(dout, filt, in_hw, c, h, w, n, *, stride=1, pad=0, alpha=1.0):
    """(value, abs_sum) of one element of din in fp64."""
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    filt = np.ascontiguousarray(filt, dtype=np.float32)
    No, Ho, Wo, Nb = dout.shape
    Nc, Sk, _, _ = filt.shape
    d = _desc(Nb, in_hw[1], in_hw[0], Nc, No, Sk, stride, pad, alpha)
    a = ctypes.c_double()
    v = _load().oracle_conv_bprop_data_point(ctypes.byref(d), dout.ctypes.data, filt.ctypes.data,
                                             int(c), int(h), int(w), int(n), ctypes.byref(a))
    return float(v), float(a.value)


def conv_bprop_filter(inp, dout, Sk, *, stride=1, pad=0, alpha=1.0, nthreads=0):
    """dfilt[Nc,Sk,Sk,No] from in[Nc,Hi,Wi,Nb] and dout[No,Ho,Wo,Nb].

    The adjoint of FPROP with respect to the filters, alpha included.
    """
    inp = np.ascontiguousarray(inp, dtype=np.float32)
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    Nc, Hi, Wi, Nb = inp.shape
    No, Ho, Wo, Nb2 = dout.shape
    if Nb2 != Nb or out_dims(Nb, Wi, Hi, Nc, No, Sk, stride, pad) != (Ho, Wo):
        raise ValueError("maps / dout do not belong to one convolution")
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    dfilt = np.zeros((Nc, Sk, Sk, No), dtype=np.float32)
    rc = _load().oracle_conv_bprop_filter(ctypes.byref(d), inp.ctypes.data, dout.ctypes.data,
                                          dfilt.ctypes.data, int(nthreads))
    if rc:
        raise RuntimeError("oracle_conv_bprop_filter failed (%d)" % rc)
    return dfilt


def conv_bprop_filter_point(inp, dout, Sk, c, kh, kw, o, *, stride=1, pad=0, alpha=1.0):
    """(value, abs_sum) of one element of dfilt in fp64."""
    inp = np.ascontiguousarray(inp, dtype=np.float32)
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    Nc, Hi, Wi, Nb = inp.shape
    No = dout.shape[0]
    d = _desc(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha)
    a = ctypes.c_double()
    v = _load().oracle_conv_bprop_filter_point(ctypes.byref(d), inp.ctypes.data,
                                               dout.ctypes.data, int(c), int(kh), int(kw),
                                               int(o), ctypes.byref(a))
    return float(v), float(a.value)


def num_threads() -> int:
    return int(_load().oracle_num_threads())
