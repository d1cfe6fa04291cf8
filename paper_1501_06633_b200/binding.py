"""ctypes binding of ``libmaxdnn.so``: same names as ``include/maxdnn.h``,
argument marshalling only.  Tensors are torch CUDA tensors (device memory and
streams are all torch is used for); every step of the computation runs in the
library's kernels.  A missing library or a failing call raises — nothing here
falls back to another implementation."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

__all__ = [
    "MaxdnnError", "ConvDesc", "PlanInfo", "KStep", "WorkItem", "conv_plan_items", "KERNEL_FP32", "KERNEL_TF32", "KERNEL_BF16",
    "OK", "INVALID_VALUE", "NOT_SUPPORTED", "CUDA_ERROR", "DEVICE_TIMEOUT",
    "library_path", "load_library", "status_string", "conv_out_dims", "conv_flops",
    "conv_in_elems", "conv_filt_elems", "conv_out_elems", "conv_plan_query", "conv_fprop",
    "conv_fprop_tf32", "conv_fprop_bf16", "conv_fprop_host", "conv_fprop_noalloc",
    "last_device_status", "last_device_status_noalloc",
    "set_option", "unset_option", "get_option", "reset_options", "last_kernel_clock",
    "launch_count", "fprop_status", "EXPORTED_SYMBOLS",
    "conv_fprop_tf32x3_workspace", "conv_fprop_tf32x3",
    "conv_bprop_data_tf32x3_workspace", "conv_bprop_data_tf32x3",
    "conv_bprop_filter_tf32x3_workspace", "conv_bprop_filter_tf32x3",
    "ConvDesc2", "conv2_out_dims", "conv2_fprop", "conv2_fprop_status",
    "conv2_bprop_data_workspace", "conv2_bprop_data", "conv2_bprop_filter_workspace",
    "conv2_bprop_filter",
    "conv_fprop_ragged_workspace", "conv_fprop_ragged", "fprop_ragged_status",
    "conv_bprop_data_workspace", "conv_bprop_data", "bprop_data_status",
    "conv_bprop_filter_workspace", "conv_bprop_filter", "bprop_filter_status",
]

OK, INVALID_VALUE, NOT_SUPPORTED, CUDA_ERROR, DEVICE_TIMEOUT = 0, 1, 2, 3, 4
KERNEL_FP32, KERNEL_TF32, KERNEL_BF16 = 0, 1, 2

EXPORTED_SYMBOLS = [
    "maxdnn_status_string", "maxdnn_conv_out_dims", "maxdnn_conv_flops", "maxdnn_conv_in_elems",
    "maxdnn_conv_filt_elems", "maxdnn_conv_out_elems", "maxdnn_conv_plan_query",
    "maxdnn_conv_fprop", "maxdnn_conv_fprop_tf32", "maxdnn_conv_fprop_bf16",
    "maxdnn_conv_fprop_host", "maxdnn_conv_fprop_noalloc", "maxdnn_last_device_status",
    "maxdnn_launch_count", "maxdnn_conv_bprop_data_workspace", "maxdnn_conv_bprop_data",
    "maxdnn_conv_bprop_filter_workspace", "maxdnn_conv_bprop_filter",
    "maxdnn_conv_fprop_ragged_workspace", "maxdnn_conv_fprop_ragged",
    "maxdnn_conv2_out_dims", "maxdnn_conv2_fprop",
    "maxdnn_conv_fprop_tf32x3_workspace", "maxdnn_conv_fprop_tf32x3",
    "maxdnn_conv_bprop_data_tf32x3_workspace", "maxdnn_conv_bprop_data_tf32x3",
    "maxdnn_conv_bprop_filter_tf32x3_workspace", "maxdnn_conv_bprop_filter_tf32x3",
    "maxdnn_conv2_bprop_data_workspace", "maxdnn_conv2_bprop_data",
    "maxdnn_conv2_bprop_filter_workspace", "maxdnn_conv2_bprop_filter",
    "maxdnn_last_device_status_noalloc", "maxdnn_set_option", "maxdnn_unset_option",
    "maxdnn_get_option", "maxdnn_reset_options", "maxdnn_last_kernel_clock",
    "maxdnn_conv_plan_items",
]


class MaxdnnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s failed: %s" % (where, status_string(status)))


class ConvDesc(ctypes.Structure):
    """maxdnn_conv_desc: Section 2's symbols."""

    _fields_ = [
        ("Nb", ctypes.c_int32), ("Wi", ctypes.c_int32), ("Hi", ctypes.c_int32),
        ("Nc", ctypes.c_int32), ("No", ctypes.c_int32), ("Sk", ctypes.c_int32),
        ("stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("alpha", ctypes.c_float),
    ]

    @classmethod
    def make(cls, Nb, Wi, Hi, Nc, No, Sk, stride=1, pad=0, alpha=1.0) -> "ConvDesc":
        return cls(int(Nb), int(Wi), int(Hi), int(Nc), int(No), int(Sk), int(stride), int(pad),
                   float(alpha))


class ConvDesc2(ctypes.Structure):
    """maxdnn_conv_desc2: per-axis filter size, stride and padding (w before h)."""

    _fields_ = [(n, ctypes.c_int32) for n in ("Nb", "Wi", "Hi", "Nc", "No", "Skw", "Skh",
                                              "stride_w", "stride_h", "pad_w", "pad_h")] + \
               [("alpha", ctypes.c_float)]

    @classmethod
    def make(cls, Nb, Wi, Hi, Nc, No, Skw, Skh, stride_w=1, stride_h=1, pad_w=0, pad_h=0,
             alpha=1.0) -> "ConvDesc2":
        return cls(int(Nb), int(Wi), int(Hi), int(Nc), int(No), int(Skw), int(Skh), int(stride_w),
                   int(stride_h), int(pad_w), int(pad_h), float(alpha))


class KStep(ctypes.Structure):
    _fields_ = [("c0", ctypes.c_int16), ("kh", ctypes.c_int8), ("kw0", ctypes.c_int8)]


class PlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "Ho", "Wo", "tile_m", "tile_px", "tile_n", "kc", "kwc", "n_ksteps", "stages", "n_tiles",
        "grid", "smem_bytes", "tile_cols", "pair", "khc", "split_tiles")]


class WorkItem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("tile", "s0", "s1", "kind")]


_lib = None


def library_path() -> str:
    """The in-tree library, or the file named by the environment variable MAXDNN_LIBRARY
    (another build of the same sources, e.g. with different compile-time switches)."""
    override = os.environ.get("MAXDNN_LIBRARY")
    if override:
        return override
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmaxdnn.so")


def load_library():
    """Load ``libmaxdnn.so`` (built in-tree by ``paper_1501_06633_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(
            "%s is missing: build it with `python -m paper_1501_06633_b200.build` "
            "(there is no fallback implementation)" % path)
    lib = ctypes.CDLL(path)
    P = ctypes.POINTER
    vp = ctypes.c_void_p
    lib.maxdnn_status_string.restype = ctypes.c_char_p
    lib.maxdnn_status_string.argtypes = [ctypes.c_int]
    lib.maxdnn_conv_out_dims.restype = ctypes.c_int
    lib.maxdnn_conv_out_dims.argtypes = [P(ConvDesc), P(ctypes.c_int32), P(ctypes.c_int32)]
    for name in ("maxdnn_conv_flops", "maxdnn_conv_in_elems", "maxdnn_conv_filt_elems",
                 "maxdnn_conv_out_elems"):
        getattr(lib, name).restype = ctypes.c_uint64
        getattr(lib, name).argtypes = [P(ConvDesc)]
    lib.maxdnn_conv_plan_query.restype = ctypes.c_int
    lib.maxdnn_conv_plan_query.argtypes = [P(ConvDesc), ctypes.c_int, ctypes.c_int32, P(PlanInfo),
                                           P(KStep), ctypes.c_int32]
    lib.maxdnn_conv_plan_items.restype = ctypes.c_int
    lib.maxdnn_conv_plan_items.argtypes = [P(ConvDesc), ctypes.c_int32, ctypes.c_int32, P(WorkItem),
                                           ctypes.c_int32, P(ctypes.c_int32)]
    for name in ("maxdnn_conv_fprop", "maxdnn_conv_fprop_tf32", "maxdnn_conv_fprop_bf16",
                 "maxdnn_conv_fprop_noalloc"):
        getattr(lib, name).restype = ctypes.c_int
        getattr(lib, name).argtypes = [P(ConvDesc), vp, vp, vp, vp]
    lib.maxdnn_conv_fprop_host.restype = ctypes.c_int
    lib.maxdnn_conv_fprop_host.argtypes = [P(ConvDesc), ctypes.c_int, vp, vp, vp, vp, vp, vp, vp]
    lib.maxdnn_conv_fprop_tf32x3_workspace.restype = ctypes.c_int
    lib.maxdnn_conv_fprop_tf32x3_workspace.argtypes = [P(ConvDesc), P(ctypes.c_size_t)]
    lib.maxdnn_conv_fprop_tf32x3.restype = ctypes.c_int
    lib.maxdnn_conv_fprop_tf32x3.argtypes = [P(ConvDesc), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.maxdnn_conv_bprop_data_tf32x3_workspace.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_data_tf32x3_workspace.argtypes = [P(ConvDesc), P(ctypes.c_size_t)]
    lib.maxdnn_conv_bprop_data_tf32x3.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_data_tf32x3.argtypes = [P(ConvDesc), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.maxdnn_conv_bprop_filter_tf32x3_workspace.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_filter_tf32x3_workspace.argtypes = [P(ConvDesc), P(ctypes.c_size_t)]
    lib.maxdnn_conv_bprop_filter_tf32x3.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_filter_tf32x3.argtypes = [P(ConvDesc), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.maxdnn_conv2_out_dims.restype = ctypes.c_int
    lib.maxdnn_conv2_out_dims.argtypes = [P(ConvDesc2), P(ctypes.c_int32), P(ctypes.c_int32)]
    lib.maxdnn_conv2_fprop.restype = ctypes.c_int
    lib.maxdnn_conv2_fprop.argtypes = [P(ConvDesc2), ctypes.c_int, vp, vp, vp, vp]
    for name in ("maxdnn_conv2_bprop_data_workspace", "maxdnn_conv2_bprop_filter_workspace"):
        getattr(lib, name).restype = ctypes.c_int
        getattr(lib, name).argtypes = [P(ConvDesc2), ctypes.c_int, P(ctypes.c_size_t)]
    for name in ("maxdnn_conv2_bprop_data", "maxdnn_conv2_bprop_filter"):
        getattr(lib, name).restype = ctypes.c_int
        getattr(lib, name).argtypes = [P(ConvDesc2), ctypes.c_int, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.maxdnn_conv_fprop_ragged_workspace.restype = ctypes.c_int
    lib.maxdnn_conv_fprop_ragged_workspace.argtypes = [P(ConvDesc), ctypes.c_int, P(ctypes.c_size_t)]
    lib.maxdnn_conv_fprop_ragged.restype = ctypes.c_int
    lib.maxdnn_conv_fprop_ragged.argtypes = [P(ConvDesc), ctypes.c_int, vp, vp, vp, vp,
                                             ctypes.c_size_t, vp]
    lib.maxdnn_conv_bprop_data_workspace.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_data_workspace.argtypes = [P(ConvDesc), ctypes.c_int, P(ctypes.c_size_t)]
    lib.maxdnn_conv_bprop_data.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_data.argtypes = [P(ConvDesc), ctypes.c_int, vp, vp, vp, vp,
                                           ctypes.c_size_t, vp]
    lib.maxdnn_conv_bprop_filter_workspace.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_filter_workspace.argtypes = [P(ConvDesc), ctypes.c_int, P(ctypes.c_size_t)]
    lib.maxdnn_conv_bprop_filter.restype = ctypes.c_int
    lib.maxdnn_conv_bprop_filter.argtypes = [P(ConvDesc), ctypes.c_int, vp, vp, vp, vp,
                                             ctypes.c_size_t, vp]
    lib.maxdnn_last_device_status.restype = ctypes.c_int
    lib.maxdnn_last_device_status.argtypes = [vp]
    lib.maxdnn_last_device_status_noalloc.restype = ctypes.c_int
    lib.maxdnn_last_device_status_noalloc.argtypes = [vp]
    lib.maxdnn_set_option.restype = ctypes.c_int
    lib.maxdnn_set_option.argtypes = [ctypes.c_char_p, ctypes.c_int32]
    lib.maxdnn_unset_option.restype = ctypes.c_int
    lib.maxdnn_unset_option.argtypes = [ctypes.c_char_p]
    lib.maxdnn_get_option.restype = ctypes.c_int
    lib.maxdnn_get_option.argtypes = [ctypes.c_char_p, P(ctypes.c_int32), P(ctypes.c_int32)]
    lib.maxdnn_last_kernel_clock.restype = ctypes.c_int
    lib.maxdnn_last_kernel_clock.argtypes = [P(ctypes.c_uint32), P(ctypes.c_uint32), vp]
    lib.maxdnn_reset_options.restype = None
    lib.maxdnn_reset_options.argtypes = []
    lib.maxdnn_launch_count.restype = ctypes.c_uint64
    lib.maxdnn_launch_count.argtypes = []
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().maxdnn_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise MaxdnnError(status, where)


def conv_out_dims(desc: ConvDesc):
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().maxdnn_conv_out_dims(ctypes.byref(desc), ctypes.byref(ho),
                                               ctypes.byref(wo)), "maxdnn_conv_out_dims")
    return ho.value, wo.value


def conv_flops(desc: ConvDesc) -> int:
    return int(load_library().maxdnn_conv_flops(ctypes.byref(desc)))


def conv_in_elems(desc: ConvDesc) -> int:
    return int(load_library().maxdnn_conv_in_elems(ctypes.byref(desc)))


def conv_filt_elems(desc: ConvDesc) -> int:
    return int(load_library().maxdnn_conv_filt_elems(ctypes.byref(desc)))


def conv_out_elems(desc: ConvDesc) -> int:
    return int(load_library().maxdnn_conv_out_elems(ctypes.byref(desc)))


def conv_plan_query(desc: ConvDesc, kind: int = KERNEL_FP32, sm_count: int = 148):
    """(PlanInfo, [KStep...]) — host-only; needs no GPU when sm_count > 0."""
    info = PlanInfo()
    steps = (KStep * 1024)()
    _check(load_library().maxdnn_conv_plan_query(ctypes.byref(desc), int(kind), int(sm_count),
                                                 ctypes.byref(info), steps, 1024),
           "maxdnn_conv_plan_query")
    return info, [steps[i] for i in range(info.n_ksteps)]


def conv_plan_items(desc: ConvDesc, cta: int, sm_count: int = 148):
    """The work items [(tile, s0, s1, kind)...] of one CTA of the fp32 kernel's plan."""
    items = (WorkItem * 4096)()
    n = ctypes.c_int32(0)
    _check(load_library().maxdnn_conv_plan_items(ctypes.byref(desc), int(sm_count), int(cta), items,
                                                 4096, ctypes.byref(n)), "maxdnn_conv_plan_items")
    return [(items[i].tile, items[i].s0, items[i].s1, items[i].kind) for i in range(min(n.value, 4096))]


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(int(stream.cuda_stream))


def _dev_ptr(t, dtype_names, n_elems, what):
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor" % what)
    if str(t.dtype).replace("torch.", "") not in dtype_names:
        raise TypeError("%s has dtype %s, expected one of %s" % (what, t.dtype, dtype_names))
    if t.numel() != n_elems:
        raise ValueError("%s has %d elements, expected %d" % (what, t.numel(), n_elems))
    return ctypes.c_void_p(t.data_ptr())


def fprop_status(desc: ConvDesc, inp, filt, out, kind: int = KERNEL_FP32, stream=None) -> int:
    """Enqueue one FPROP on torch tensors and return the raw status code."""
    lib = load_library()
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pin = _dev_ptr(inp, in_types, conv_in_elems(desc), "in")
    pf = _dev_ptr(filt, in_types, conv_filt_elems(desc), "filt")
    po = _dev_ptr(out, ("float32",), conv_out_elems(desc), "out")
    fn = {KERNEL_FP32: lib.maxdnn_conv_fprop, KERNEL_TF32: lib.maxdnn_conv_fprop_tf32,
          KERNEL_BF16: lib.maxdnn_conv_fprop_bf16}[kind]
    return int(fn(ctypes.byref(desc), pin, pf, po, _stream_ptr(stream)))


def conv_fprop(desc: ConvDesc, inp, filt, out, stream=None) -> None:
    """maxdnn_conv_fprop: exact fp32 FPROP on device tensors (asynchronous)."""
    _check(fprop_status(desc, inp, filt, out, KERNEL_FP32, stream), "maxdnn_conv_fprop")


def conv_fprop_noalloc(desc: ConvDesc, inp, filt, out, stream=None) -> None:
    """maxdnn_conv_fprop_noalloc: the fp32 FPROP for callers that must not
    allocate — the library itself makes no allocation call on this path (its
    status block is a device array built into the library).  Tensors are the
    caller's, as for conv_fprop; calls that overlap on the GPU race on the
    shared block."""
    lib = load_library()
    pin = _dev_ptr(inp, ("float32",), conv_in_elems(desc), "in")
    pf = _dev_ptr(filt, ("float32",), conv_filt_elems(desc), "filt")
    po = _dev_ptr(out, ("float32",), conv_out_elems(desc), "out")
    _check(int(lib.maxdnn_conv_fprop_noalloc(ctypes.byref(desc), pin, pf, po, _stream_ptr(stream))),
           "maxdnn_conv_fprop_noalloc")


def conv_fprop_tf32(desc: ConvDesc, inp, filt, out, stream=None) -> None:
    _check(fprop_status(desc, inp, filt, out, KERNEL_TF32, stream), "maxdnn_conv_fprop_tf32")


def conv_fprop_bf16(desc: ConvDesc, inp, filt, out, stream=None) -> None:
    _check(fprop_status(desc, inp, filt, out, KERNEL_BF16, stream), "maxdnn_conv_fprop_bf16")


def conv_fprop_host(desc: ConvDesc, kind: int, h_in, h_filt, h_out, d_in, d_filt, d_out,
                    stream=None) -> None:
    """maxdnn_conv_fprop_host: h_* are CPU (ideally pinned) tensors, d_* device
    staging tensors of the same sizes; copies and kernel are enqueued on the stream."""
    import torch
    for t, what in ((h_in, "h_in"), (h_filt, "h_filt"), (h_out, "h_out")):
        if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.is_contiguous()):
            raise TypeError("%s must be a contiguous CPU tensor" % what)
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pin = _dev_ptr(d_in, in_types, conv_in_elems(desc), "d_in")
    pf = _dev_ptr(d_filt, in_types, conv_filt_elems(desc), "d_filt")
    po = _dev_ptr(d_out, ("float32",), conv_out_elems(desc), "d_out")
    if h_in.numel() != d_in.numel() or h_filt.numel() != d_filt.numel() or \
            h_out.numel() != d_out.numel() or h_in.element_size() != d_in.element_size() or \
            h_filt.element_size() != d_filt.element_size() or h_out.dtype != torch.float32:
        raise ValueError("host and device buffers do not match")
    _check(load_library().maxdnn_conv_fprop_host(
        ctypes.byref(desc), int(kind), ctypes.c_void_p(h_in.data_ptr()),
        ctypes.c_void_p(h_filt.data_ptr()), ctypes.c_void_p(h_out.data_ptr()), pin, pf, po,
        _stream_ptr(stream)), "maxdnn_conv_fprop_host")


def _workspace_ptr(workspace, need):
    import torch
    if workspace is None:
        if need:
            raise ValueError("this call needs %d bytes of device workspace" % need)
        return ctypes.c_void_p(0), 0
    if not (isinstance(workspace, torch.Tensor) and workspace.is_cuda and workspace.is_contiguous()):
        raise TypeError("workspace must be a contiguous CUDA tensor")
    return ctypes.c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size()


def conv_fprop_tf32x3_workspace(desc: ConvDesc) -> int:
    """Bytes of device scratch maxdnn_conv_fprop_tf32x3 needs (the split maps and filters)."""
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv_fprop_tf32x3_workspace(ctypes.byref(desc),
                                                                 ctypes.byref(n))),
           "maxdnn_conv_fprop_tf32x3_workspace")
    return int(n.value)


def conv_fprop_tf32x3(desc: ConvDesc, inp, filt, out, workspace, stream=None) -> None:
    """maxdnn_conv_fprop_tf32x3: fp32-level accuracy on the tensor cores (three TF32 products)."""
    lib = load_library()
    pin = _dev_ptr(inp, ("float32",), conv_in_elems(desc), "in")
    pf = _dev_ptr(filt, ("float32",), conv_filt_elems(desc), "filt")
    po = _dev_ptr(out, ("float32",), conv_out_elems(desc), "out")
    pw, nbytes = _workspace_ptr(workspace, 1)
    _check(int(lib.maxdnn_conv_fprop_tf32x3(ctypes.byref(desc), pin, pf, po, pw, nbytes,
                                            _stream_ptr(stream))), "maxdnn_conv_fprop_tf32x3")


def conv_bprop_data_tf32x3_workspace(desc: ConvDesc) -> int:
    """Bytes of device scratch maxdnn_conv_bprop_data_tf32x3 needs."""
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv_bprop_data_tf32x3_workspace(ctypes.byref(desc),
                                                                      ctypes.byref(n))),
           "maxdnn_conv_bprop_data_tf32x3_workspace")
    return int(n.value)


def conv_bprop_data_tf32x3(desc: ConvDesc, dout, filt, din, workspace, stream=None) -> None:
    """maxdnn_conv_bprop_data_tf32x3: map gradient (stride 1) in the three-product TF32 mode."""
    lib = load_library()
    pg = _dev_ptr(dout, ("float32",), conv_out_elems(desc), "dout")
    pf = _dev_ptr(filt, ("float32",), conv_filt_elems(desc), "filt")
    px = _dev_ptr(din, ("float32",), conv_in_elems(desc), "din")
    pw, nbytes = _workspace_ptr(workspace, 1)
    _check(int(lib.maxdnn_conv_bprop_data_tf32x3(ctypes.byref(desc), pg, pf, px, pw, nbytes,
                                                 _stream_ptr(stream))),
           "maxdnn_conv_bprop_data_tf32x3")


def conv_bprop_filter_tf32x3_workspace(desc: ConvDesc) -> int:
    """Bytes of device scratch maxdnn_conv_bprop_filter_tf32x3 needs."""
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv_bprop_filter_tf32x3_workspace(ctypes.byref(desc),
                                                                        ctypes.byref(n))),
           "maxdnn_conv_bprop_filter_tf32x3_workspace")
    return int(n.value)


def conv_bprop_filter_tf32x3(desc: ConvDesc, inp, dout, dfilt, workspace, stream=None) -> None:
    """maxdnn_conv_bprop_filter_tf32x3: filter gradient in the three-product TF32 mode."""
    lib = load_library()
    px = _dev_ptr(inp, ("float32",), conv_in_elems(desc), "in")
    pg = _dev_ptr(dout, ("float32",), conv_out_elems(desc), "dout")
    pf = _dev_ptr(dfilt, ("float32",), conv_filt_elems(desc), "dfilt")
    pw, nbytes = _workspace_ptr(workspace, 1)
    _check(int(lib.maxdnn_conv_bprop_filter_tf32x3(ctypes.byref(desc), px, pg, pf, pw, nbytes,
                                                   _stream_ptr(stream))),
           "maxdnn_conv_bprop_filter_tf32x3")


def conv2_out_dims(desc: ConvDesc2):
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    _check(int(load_library().maxdnn_conv2_out_dims(ctypes.byref(desc), ctypes.byref(ho),
                                                     ctypes.byref(wo))), "maxdnn_conv2_out_dims")
    return ho.value, wo.value


def conv2_fprop_status(desc: ConvDesc2, inp, filt, out, kind: int = KERNEL_FP32, stream=None) -> int:
    """Enqueue maxdnn_conv2_fprop on torch tensors; returns the raw status code."""
    lib = load_library()
    Ho, Wo = conv2_out_dims(desc)
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pin = _dev_ptr(inp, in_types, desc.Nc * desc.Hi * desc.Wi * desc.Nb, "in")
    pf = _dev_ptr(filt, in_types, desc.Nc * desc.Skh * desc.Skw * desc.No, "filt")
    po = _dev_ptr(out, ("float32",), desc.No * Ho * Wo * desc.Nb, "out")
    return int(lib.maxdnn_conv2_fprop(ctypes.byref(desc), int(kind), pin, pf, po,
                                      _stream_ptr(stream)))


def conv2_fprop(desc: ConvDesc2, inp, filt, out, kind: int = KERNEL_FP32, stream=None) -> None:
    """maxdnn_conv2_fprop: FPROP with per-axis filter size, stride and padding."""
    _check(conv2_fprop_status(desc, inp, filt, out, kind, stream), "maxdnn_conv2_fprop")


def _conv2_sizes(desc: ConvDesc2):
    Ho, Wo = conv2_out_dims(desc)
    return (desc.Nc * desc.Hi * desc.Wi * desc.Nb, desc.Nc * desc.Skh * desc.Skw * desc.No,
            desc.No * Ho * Wo * desc.Nb)


def conv2_bprop_data_workspace(desc: ConvDesc2, kind: int = KERNEL_FP32) -> int:
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv2_bprop_data_workspace(ctypes.byref(desc), int(kind),
                                                                ctypes.byref(n))),
           "maxdnn_conv2_bprop_data_workspace")
    return int(n.value)


def conv2_bprop_data(desc: ConvDesc2, dout, filt, din, workspace, kind: int = KERNEL_FP32,
                     stream=None) -> None:
    """maxdnn_conv2_bprop_data: map gradient of the per-axis operation."""
    n_in, n_f, n_out = _conv2_sizes(desc)
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pg = _dev_ptr(dout, in_types, n_out, "dout")
    pf = _dev_ptr(filt, in_types, n_f, "filt")
    pd = _dev_ptr(din, ("float32",), n_in, "din")
    pw, nbytes = _workspace_ptr(workspace, 1)
    _check(int(load_library().maxdnn_conv2_bprop_data(ctypes.byref(desc), int(kind), pg, pf, pd, pw,
                                                      nbytes, _stream_ptr(stream))),
           "maxdnn_conv2_bprop_data")


def conv2_bprop_filter_workspace(desc: ConvDesc2, kind: int = KERNEL_FP32) -> int:
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv2_bprop_filter_workspace(ctypes.byref(desc), int(kind),
                                                                  ctypes.byref(n))),
           "maxdnn_conv2_bprop_filter_workspace")
    return int(n.value)


def conv2_bprop_filter(desc: ConvDesc2, inp, dout, dfilt, workspace, kind: int = KERNEL_FP32,
                       stream=None) -> None:
    """maxdnn_conv2_bprop_filter: filter gradient of the per-axis operation."""
    n_in, n_f, n_out = _conv2_sizes(desc)
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pi = _dev_ptr(inp, in_types, n_in, "in")
    pg = _dev_ptr(dout, in_types, n_out, "dout")
    pd = _dev_ptr(dfilt, ("float32",), n_f, "dfilt")
    pw, nbytes = _workspace_ptr(workspace, 0)
    _check(int(load_library().maxdnn_conv2_bprop_filter(ctypes.byref(desc), int(kind), pi, pg, pd,
                                                        pw, nbytes, _stream_ptr(stream))),
           "maxdnn_conv2_bprop_filter")


def conv_fprop_ragged_workspace(desc: ConvDesc, kind: int = KERNEL_FP32) -> int:
    """Bytes of device scratch maxdnn_conv_fprop_ragged needs (0: the shape needs no padding)."""
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv_fprop_ragged_workspace(ctypes.byref(desc), int(kind),
                                                                 ctypes.byref(n))),
           "maxdnn_conv_fprop_ragged_workspace")
    return int(n.value)


def fprop_ragged_status(desc: ConvDesc, inp, filt, out, workspace, kind: int = KERNEL_FP32,
                        stream=None) -> int:
    """Enqueue maxdnn_conv_fprop_ragged on torch tensors; returns the raw status code."""
    lib = load_library()
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pin = _dev_ptr(inp, in_types, conv_in_elems(desc), "in")
    pf = _dev_ptr(filt, in_types, conv_filt_elems(desc), "filt")
    po = _dev_ptr(out, ("float32",), conv_out_elems(desc), "out")
    pw, nbytes = _workspace_ptr(workspace, 0)
    return int(lib.maxdnn_conv_fprop_ragged(ctypes.byref(desc), int(kind), pin, pf, po, pw, nbytes,
                                            _stream_ptr(stream)))


def conv_fprop_ragged(desc: ConvDesc, inp, filt, out, workspace, kind: int = KERNEL_FP32,
                      stream=None) -> None:
    """maxdnn_conv_fprop_ragged: FPROP for any Nb / No, through zero-padded staging tensors."""
    _check(fprop_ragged_status(desc, inp, filt, out, workspace, kind, stream),
           "maxdnn_conv_fprop_ragged")


def conv_bprop_data_workspace(desc: ConvDesc, kind: int = KERNEL_FP32) -> int:
    """Bytes of device scratch maxdnn_conv_bprop_data needs (the transformed filter bank)."""
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv_bprop_data_workspace(ctypes.byref(desc), int(kind),
                                                               ctypes.byref(n))),
           "maxdnn_conv_bprop_data_workspace")
    return int(n.value)


def bprop_data_status(desc: ConvDesc, dout, filt, din, workspace, kind: int = KERNEL_FP32,
                      stream=None) -> int:
    """Enqueue maxdnn_conv_bprop_data on torch tensors; returns the raw status code."""
    lib = load_library()
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pg = _dev_ptr(dout, in_types, conv_out_elems(desc), "dout")
    pf = _dev_ptr(filt, in_types, conv_filt_elems(desc), "filt")
    pd = _dev_ptr(din, ("float32",), conv_in_elems(desc), "din")
    pw, nbytes = _workspace_ptr(workspace, 1)
    return int(lib.maxdnn_conv_bprop_data(ctypes.byref(desc), int(kind), pg, pf, pd, pw, nbytes,
                                          _stream_ptr(stream)))


def conv_bprop_data(desc: ConvDesc, dout, filt, din, workspace, kind: int = KERNEL_FP32,
                    stream=None) -> None:
    """maxdnn_conv_bprop_data: gradient with respect to the maps (asynchronous)."""
    _check(bprop_data_status(desc, dout, filt, din, workspace, kind, stream),
           "maxdnn_conv_bprop_data")


def conv_bprop_filter_workspace(desc: ConvDesc, kind: int = KERNEL_FP32) -> int:
    """Bytes of device scratch maxdnn_conv_bprop_filter needs (partial sums; may be 0)."""
    n = ctypes.c_size_t()
    _check(int(load_library().maxdnn_conv_bprop_filter_workspace(ctypes.byref(desc), int(kind),
                                                                 ctypes.byref(n))),
           "maxdnn_conv_bprop_filter_workspace")
    return int(n.value)


def bprop_filter_status(desc: ConvDesc, inp, dout, dfilt, workspace, kind: int = KERNEL_FP32,
                        stream=None) -> int:
    """Enqueue maxdnn_conv_bprop_filter on torch tensors; returns the raw status code."""
    lib = load_library()
    in_types = ("bfloat16", "uint16", "int16") if kind == KERNEL_BF16 else ("float32",)
    pi = _dev_ptr(inp, in_types, conv_in_elems(desc), "in")
    pg = _dev_ptr(dout, in_types, conv_out_elems(desc), "dout")
    pd = _dev_ptr(dfilt, ("float32",), conv_filt_elems(desc), "dfilt")
    pw, nbytes = _workspace_ptr(workspace, 0)
    return int(lib.maxdnn_conv_bprop_filter(ctypes.byref(desc), int(kind), pi, pg, pd, pw, nbytes,
                                            _stream_ptr(stream)))


def conv_bprop_filter(desc: ConvDesc, inp, dout, dfilt, workspace, kind: int = KERNEL_FP32,
                      stream=None) -> None:
    """maxdnn_conv_bprop_filter: gradient with respect to the filters (fp32 / tf32 / bf16)."""
    _check(bprop_filter_status(desc, inp, dout, dfilt, workspace, kind, stream),
           "maxdnn_conv_bprop_filter")


def last_device_status(stream=None) -> int:
    return int(load_library().maxdnn_last_device_status(_stream_ptr(stream)))


def last_device_status_noalloc(stream=None) -> int:
    return int(load_library().maxdnn_last_device_status_noalloc(_stream_ptr(stream)))


def set_option(name: str, value: int) -> None:
    st = load_library().maxdnn_set_option(name.encode(), int(value))
    if st != OK:
        raise MaxdnnError(st, "maxdnn_set_option(%s)" % name)


def unset_option(name: str) -> None:
    st = load_library().maxdnn_unset_option(name.encode())
    if st != OK:
        raise MaxdnnError(st, "maxdnn_unset_option(%s)" % name)


def get_option(name: str):
    """(value, is_set) of a tuning option."""
    v, isset = ctypes.c_int32(0), ctypes.c_int32(0)
    st = load_library().maxdnn_get_option(name.encode(), ctypes.byref(v), ctypes.byref(isset))
    if st != OK:
        raise MaxdnnError(st, "maxdnn_get_option(%s)" % name)
    return int(v.value), bool(isset.value)


def last_kernel_clock(stream=None):
    """(sm_cycles, nanoseconds) of the latest fp32 FPROP launch made with option KERNEL_CLOCK."""
    c, ns = ctypes.c_uint32(0), ctypes.c_uint32(0)
    st = load_library().maxdnn_last_kernel_clock(ctypes.byref(c), ctypes.byref(ns), _stream_ptr(stream))
    if st != OK:
        raise MaxdnnError(st, "maxdnn_last_kernel_clock")
    return int(c.value), int(ns.value)


def reset_options() -> None:
    load_library().maxdnn_reset_options()


def launch_count() -> int:
    return int(load_library().maxdnn_launch_count())
