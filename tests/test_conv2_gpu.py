"""FPROP with per-axis filter size, stride and padding (rectangular filters), all three
kernels, against the per-axis oracle."""
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
    # Nb Wi Hi Nc No Skw Skh sw sh pw ph alpha
    (64, 14, 9, 32, 64, 3, 1, 1, 1, 1, 0, 1.0),       # 1 x 3 row filter
    (64, 9, 14, 32, 64, 1, 3, 1, 1, 0, 1, 1.0),       # 3 x 1 column filter
    (128, 12, 10, 48, 96, 5, 3, 1, 1, 2, 1, 0.5),     # 3 x 5, strip reuse over 5 columns
    (64, 17, 13, 24, 160, 3, 5, 2, 1, 1, 2, 1.0),     # stride 2 across, 1 down
    (64, 16, 21, 16, 32, 4, 2, 1, 3, 0, 1, 1.0),      # stride 3 down only, even sizes
    (64, 23, 19, 3, 64, 7, 11, 4, 2, 3, 0, 1.0),      # few channels: columns merged into K (tensor)
    (64, 11, 11, 64, 256, 3, 3, 1, 1, 1, 1, 1.0),     # square through the general entry point
]


@pytest.mark.parametrize("kernel", ["fp32", "tf32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_conv2_fprop(kernel, shape):
    Nb, Wi, Hi, Nc, No, Skw, Skh, sw, sh, pw, ph, alpha = shape
    rng = np.random.default_rng(6100 + Skw * 13 + Skh)
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = rng.uniform(-1, 1, size=(Nc, Skh, Skw, No)).astype(np.float32)
    d = mx.ConvDesc2.make(Nb, Wi, Hi, Nc, No, Skw, Skh, sw, sh, pw, ph, alpha)
    if kernel == "bf16":
        to_dev = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        r_in, r_f = wl.from_bf16_bits(wl.to_bf16_bits(inp)), wl.from_bf16_bits(wl.to_bf16_bits(filt))
    else:
        to_dev = lambda a: torch.from_numpy(a).cuda()
        r_in, r_f = inp, filt
    ref = oracle.conv2_fprop(r_in, r_f, stride=(sh, sw), pad=(ph, pw), alpha=alpha)
    assert mx.conv2_out_dims(d) == ref.shape[1:3]
    out = torch.full((ref.size,), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv2_fprop(d, to_dev(inp), to_dev(filt), out, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    got = out.cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    err = float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref)))
    assert err <= TOL[kernel]
