"""Failure detection without a GPU fault: every wait inside the kernels has a time
limit; a test hook makes one CTA's barriers expect an arrival that never comes, the waiting
warps give up after their
limit, the kernel ends normally, the status word says so, and the context stays usable."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _tensors(w, kernel):
    inp, filt = wl.make_inputs(w)
    if kernel == "bf16":
        to_dev = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        ref_in, ref_f = wl.from_bf16_bits(wl.to_bf16_bits(inp)), wl.from_bf16_bits(wl.to_bf16_bits(filt))
    else:
        to_dev = lambda a: torch.from_numpy(a).cuda()
        ref_in, ref_f = inp, filt
    return to_dev(inp), to_dev(filt), ref_in, ref_f


@pytest.mark.parametrize("kernel,kind,No", [("fp32", mx.KERNEL_FP32, 128), ("bf16", mx.KERNEL_BF16, 128),
                                            ("bf16", mx.KERNEL_BF16, 256)],
                         ids=["fp32", "bf16-one-sm", "bf16-two-sm"])
def test_a_wait_that_runs_out_is_reported_and_the_context_survives(kernel, kind, No, monkeypatch):
    w = wl.WORKLOADS["large3x3"].scaled(Nb=64, Wi=12, Hi=8, Nc=64, No=No)
    d = mx.ConvDesc.make(*w.dims)
    if kernel != "fp32":
        assert mx.conv_plan_query(d, kind, 148)[0].tile_m == (256 if No == 256 else 128)
    d_in, d_f, ref_in, ref_f = _tensors(w, kernel)
    out = torch.zeros(mx.conv_out_elems(d), dtype=torch.float32, device="cuda")
    assert mx.last_device_status() == mx.OK

    mx.set_option("TEST_MISSING_ARRIVAL", 1)     # CTA 0 waits for an arrival that never comes
    assert mx.fprop_status(d, d_in, d_f, out, kind) == mx.OK          # the launch itself succeeds
    assert mx.last_device_status() == mx.DEVICE_TIMEOUT               # ...the kernel gave up waiting
    assert mx.last_device_status() == mx.OK                           # reading clears the word

    mx.unset_option("TEST_MISSING_ARRIVAL")
    assert mx.fprop_status(d, d_in, d_f, out, kind) == mx.OK          # same context, next call
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_fprop(ref_in, ref_f, stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = out.cpu().numpy().reshape(ref.shape)
    err = float(np.max(np.abs(got - ref))) / float(np.max(np.abs(ref)))
    assert err <= 1e-5


@pytest.mark.parametrize("No", [128, 256], ids=["one-sm", "two-sm"])
def test_chunked_kernel_wait_runs_out_and_the_context_survives(No, monkeypatch):
    """The same for the chunked TF32 kernels behind maxdnn_conv_fprop_tf32x3 (eight epilogue
    warps per CTA that wait for one chunk's accumulator after another)."""
    w = wl.WORKLOADS["large3x3"].scaled(Nb=64, Wi=12, Hi=8, Nc=64, No=No)
    d = mx.ConvDesc.make(*w.dims)
    inp, filt = wl.make_inputs(w)
    x, f = torch.from_numpy(inp).cuda(), torch.from_numpy(filt).cuda()
    ws = torch.empty(mx.conv_fprop_tf32x3_workspace(d), dtype=torch.uint8, device="cuda")
    out = torch.zeros(mx.conv_out_elems(d), dtype=torch.float32, device="cuda")
    assert mx.last_device_status() == mx.OK
    mx.set_option("TEST_MISSING_ARRIVAL", 1)
    mx.conv_fprop_tf32x3(d, x, f, out, ws)
    assert mx.last_device_status() == mx.DEVICE_TIMEOUT
    assert mx.last_device_status() == mx.OK
    mx.unset_option("TEST_MISSING_ARRIVAL")
    mx.conv_fprop_tf32x3(d, x, f, out, ws)
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = out.cpu().numpy().reshape(ref.shape)
    assert float(np.max(np.abs(got - ref))) / float(np.max(np.abs(ref))) <= 1e-5


@pytest.mark.parametrize("kernel,kind", [("fp32", mx.KERNEL_FP32), ("bf16", mx.KERNEL_BF16)])
def test_a_stale_timeout_code_does_not_disturb_later_launches(kernel, kind):
    """The status word is sticky until it is read.  A launch that follows a timed-out one
    WITHOUT the word having been read must still be exact: its waits leave early only for
    a give-up of their own launch (each launch carries its own number)."""
    w = wl.WORKLOADS["large3x3"].scaled(Nb=64, Wi=12, Hi=8, Nc=64, No=128)
    d = mx.ConvDesc.make(*w.dims)
    d_in, d_f, ref_in, ref_f = _tensors(w, kernel)
    bad = torch.zeros(mx.conv_out_elems(d), dtype=torch.float32, device="cuda")
    out = torch.zeros(mx.conv_out_elems(d), dtype=torch.float32, device="cuda")
    assert mx.last_device_status() == mx.OK
    mx.set_option("TEST_MISSING_ARRIVAL", 1)
    assert mx.fprop_status(d, d_in, d_f, bad, kind) == mx.OK       # this one gives up
    mx.unset_option("TEST_MISSING_ARRIVAL")
    for _ in range(3):                                                  # these must not
        assert mx.fprop_status(d, d_in, d_f, out, kind) == mx.OK
    torch.cuda.synchronize()
    ref = oracle.conv_fprop(ref_in, ref_f, stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = out.cpu().numpy().reshape(ref.shape)
    assert float(np.max(np.abs(got - ref))) / float(np.max(np.abs(ref))) <= 1e-5
    assert mx.last_device_status() == mx.DEVICE_TIMEOUT               # the code is still there
    assert mx.last_device_status() == mx.OK
