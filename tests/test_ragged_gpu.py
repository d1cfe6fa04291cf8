"""FPROP for minibatch / filter counts outside the 16-byte row rule of the bulk tensor
copies — staged inside the fp32 kernel by copy warps, through zero-padded staging tensors
for the tensor-core kernels (and for fp32 on request) — against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu

KIND = {"fp32": mx.KERNEL_FP32, "tf32": mx.KERNEL_TF32, "bf16": mx.KERNEL_BF16}
TOL = {"fp32": 1e-5, "tf32": 5e-3, "bf16": 2e-2}

SHAPES = [
    # Nb Wi Hi Nc No Sk stride pad alpha
    (30, 14, 9, 16, 50, 3, 1, 1, 1.0),       # both ragged
    (62, 20, 13, 40, 130, 3, 1, 1, 1.0),     # several tiles of 128 filters, two pixels x 64 images
    (150, 9, 7, 12, 70, 5, 1, 2, -1.0),      # two image chunks, the second ragged
    (7, 12, 12, 5, 3, 5, 2, 2, 0.5),         # tiny odd counts, stride 2
    (33, 23, 19, 3, 96, 11, 4, 0, 1.0),      # one image over a multiple of 32
    (64, 10, 8, 24, 45, 3, 1, 0, 1.0),       # only the filters ragged
    (1, 9, 9, 8, 8, 3, 1, 1, 2.0),           # a single image
]


@pytest.mark.parametrize("kernel", ["fp32", "fp32-padded", "tf32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_fprop_ragged(kernel, shape):
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    in_kernel = kernel == "fp32"
    if kernel.startswith("fp32"):
        mx.set_option("RAGGED_PADDED", -1 if in_kernel else 1)      # pin the route
        kernel = "fp32"
    w = wl.Workload("ragged", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 5150 + Nb)
    inp, filt = wl.make_inputs(w)
    d = mx.ConvDesc.make(*w.dims)
    if kernel == "fp32" and (Nb % 4 or No % 4):
        out0 = torch.empty(mx.conv_out_elems(d), dtype=torch.float32, device="cuda")
        st = mx.fprop_status(d, torch.from_numpy(inp).cuda(), torch.from_numpy(filt).cuda(), out0)
        assert st == mx.NOT_SUPPORTED                               # the plain entry point refuses
    need = mx.conv_fprop_ragged_workspace(d, KIND[kernel])
    assert (need == 0) if in_kernel else (need > 0)      # the fp32 kernel pads nothing
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    launches = mx.launch_count()
    if kernel == "bf16":
        to_dev = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        r_in, r_f = wl.from_bf16_bits(wl.to_bf16_bits(inp)), wl.from_bf16_bits(wl.to_bf16_bits(filt))
    else:
        to_dev = lambda a: torch.from_numpy(a).cuda()
        r_in, r_f = inp, filt
    out = torch.full((mx.conv_out_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_fprop_ragged(d, to_dev(inp), to_dev(filt), out, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    assert mx.launch_count() - launches == (1 if in_kernel else 4)
    ref = oracle.conv_fprop(r_in, r_f, stride=stride, pad=pad, alpha=alpha)
    got = out.cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    err = float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref)))
    assert err <= TOL[kernel]


def test_aligned_shape_needs_no_workspace_and_matches_the_plain_entry_point():
    w = wl.WORKLOADS["tiny3x3"]
    inp, filt = wl.make_inputs(w)
    d = mx.ConvDesc.make(*w.dims)
    assert mx.conv_fprop_ragged_workspace(d) == 0
    x, f = torch.from_numpy(inp).cuda(), torch.from_numpy(filt).cuda()
    a = torch.empty(mx.conv_out_elems(d), device="cuda")
    b = torch.empty_like(a)
    mx.conv_fprop(d, x, f, a)
    mx.conv_fprop_ragged(d, x, f, b, None)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    short = torch.empty(64, dtype=torch.uint8, device="cuda")
    d2 = mx.ConvDesc.make(30, 8, 8, 4, 4, 3, 1, 1, 1.0)
    x2 = torch.zeros(mx.conv_in_elems(d2), device="cuda")
    f2 = torch.zeros(mx.conv_filt_elems(d2), device="cuda")
    o2 = torch.zeros(mx.conv_out_elems(d2), device="cuda")
    assert mx.fprop_ragged_status(d2, x2, f2, o2, short) == mx.INVALID_VALUE
