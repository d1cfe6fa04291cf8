"""Seeded random shapes through every kernel against the oracle: small problems whose
planner choices (tile shape, strip reuse, merged filter columns, one or two SMs, 256 / 192 /
128 columns, reduction splits) vary from case to case."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu

KIND = {"fp32": mx.KERNEL_FP32, "tf32": mx.KERNEL_TF32, "bf16": mx.KERNEL_BF16}
TOL = {"fp32": 1e-5, "tf32": 5e-3, "bf16": 2e-2}


def random_shapes(kernel, count, seed):
    rng = np.random.default_rng(seed)
    nb_step = {"fp32": 4, "tf32": 32, "bf16": 64}[kernel]
    no_step = 4 if kernel == "fp32" else 32
    out = []
    while len(out) < count:
        Sk = int(rng.integers(1, 8))
        stride = int(rng.integers(1, 4))
        pad = int(rng.integers(0, Sk))
        Wi = int(rng.integers(max(Sk - 2 * pad, 1), 25))
        Hi = int(rng.integers(max(Sk - 2 * pad, 1), 25))
        if Wi + 2 * pad < Sk or Hi + 2 * pad < Sk:
            continue
        Nb = nb_step * int(rng.integers(1, 160 // nb_step + 1))
        Nc = int(rng.integers(1, 71))
        No = no_step * int(rng.integers(1, 288 // no_step + 1))
        alpha = float(rng.choice([1.0, 0.5, -2.0]))
        out.append((Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha))
    return out


def operands(kernel, *arrays):
    if kernel == "bf16":
        dev = [torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16) for a in arrays]
        ref = [wl.from_bf16_bits(wl.to_bf16_bits(a)) for a in arrays]
    else:
        dev = [torch.from_numpy(a).cuda() for a in arrays]
        ref = list(arrays)
    return dev, ref


def rel(got, ref):
    return float(np.max(np.abs(got.astype(np.float64) - ref))) / max(float(np.max(np.abs(ref))), 1e-30)


@pytest.mark.parametrize("kernel", ["fp32", "tf32", "bf16"])
def test_random_shapes_forward_and_gradients(kernel):
    for i, shape in enumerate(random_shapes(kernel, 60, {"fp32": 11, "tf32": 22, "bf16": 33}[kernel])):
        Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
        w = wl.Workload("fuzz", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", -1.0, 1.0),
                        ("uniform", -1.0, 1.0), 9000 + i)
        inp, filt = wl.make_inputs(w)
        dout = wl.make_dout(w)
        d = mx.ConvDesc.make(*w.dims)
        (x, f, g), (rx, rf, rg) = operands(kernel, inp, filt, dout)
        out = torch.full((mx.conv_out_elems(d),), float("nan"), device="cuda")
        assert mx.fprop_status(d, x, f, out, KIND[kernel]) == mx.OK, shape
        ref = oracle.conv_fprop(rx, rf, stride=stride, pad=pad, alpha=alpha)
        assert rel(out.cpu().numpy().reshape(ref.shape), ref) <= TOL[kernel], ("fprop", shape)
        # filter gradient (bf16 rows of images must be multiples of 16 bytes: they are)
        need = mx.conv_bprop_filter_workspace(d, KIND[kernel])
        ws = torch.empty(max(16, need), dtype=torch.uint8, device="cuda")
        dfilt = torch.full((mx.conv_filt_elems(d),), float("nan"), device="cuda")
        assert mx.bprop_filter_status(d, x, g, dfilt, ws, KIND[kernel]) == mx.OK, ("wgrad", shape)
        ref = oracle.conv_bprop_filter(rx, rg, Sk, stride=stride, pad=pad, alpha=alpha)
        assert rel(dfilt.cpu().numpy().reshape(ref.shape), ref) <= TOL[kernel], ("wgrad", shape)
        # map gradient where the transposed problem is accepted (its filter count is Nc)
        try:
            need = mx.conv_bprop_data_workspace(d, KIND[kernel])
        except mx.MaxdnnError:
            continue
        ws = torch.empty(max(16, need), dtype=torch.uint8, device="cuda")
        din = torch.full((mx.conv_in_elems(d),), float("nan"), device="cuda")
        st = mx.bprop_data_status(d, g, f, din, ws, KIND[kernel])
        if st == mx.OK:
            ref = oracle.conv_bprop_data(rg, rf, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
            assert rel(din.cpu().numpy().reshape(ref.shape), ref) <= TOL[kernel], ("dgrad", shape)
        else:
            assert st == mx.NOT_SUPPORTED, ("dgrad", shape, st)
        assert mx.last_device_status() == mx.OK


@pytest.mark.parametrize("kernel", ["fp32", "tf32", "bf16"])
def test_random_per_axis_shapes(kernel):
    rng = np.random.default_rng({"fp32": 101, "tf32": 202, "bf16": 303}[kernel])
    nb_step = {"fp32": 4, "tf32": 32, "bf16": 64}[kernel]
    no_step = 4 if kernel == "fp32" else 32
    done = 0
    while done < 40:
        Skw, Skh = int(rng.integers(1, 8)), int(rng.integers(1, 8))
        sw, sh = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        pw, ph = int(rng.integers(0, Skw)), int(rng.integers(0, Skh))
        Wi, Hi = int(rng.integers(1, 22)), int(rng.integers(1, 22))
        if Wi + 2 * pw < Skw or Hi + 2 * ph < Skh:
            continue
        Nb = nb_step * int(rng.integers(1, 128 // nb_step + 1))
        Nc = int(rng.integers(1, 50))
        No = no_step * int(rng.integers(1, 288 // no_step + 1))
        alpha = float(rng.choice([1.0, 0.25]))
        inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
        filt = rng.uniform(-1, 1, size=(Nc, Skh, Skw, No)).astype(np.float32)
        d = mx.ConvDesc2.make(Nb, Wi, Hi, Nc, No, Skw, Skh, sw, sh, pw, ph, alpha)
        (x, f), (rx, rf) = operands(kernel, inp, filt)
        ref = oracle.conv2_fprop(rx, rf, stride=(sh, sw), pad=(ph, pw), alpha=alpha)
        out = torch.full((ref.size,), float("nan"), device="cuda")
        shape = (Nb, Wi, Hi, Nc, No, Skw, Skh, sw, sh, pw, ph)
        assert mx.conv2_fprop_status(d, x, f, out, KIND[kernel]) == mx.OK, shape
        assert rel(out.cpu().numpy().reshape(ref.shape), ref) <= TOL[kernel], shape
        # both gradients of the per-axis operation
        dout = rng.uniform(-1, 1, size=ref.shape).astype(np.float32)
        (g,), (rg,) = operands(kernel, dout)
        ws = torch.empty(max(16, mx.conv2_bprop_filter_workspace(d, KIND[kernel])), dtype=torch.uint8,
                         device="cuda")
        dfilt = torch.full((filt.size,), float("nan"), device="cuda")
        mx.conv2_bprop_filter(d, x, g, dfilt, ws, KIND[kernel])
        rdf = oracle.conv2_bprop_filter(rx, rg, (Skh, Skw), stride=(sh, sw), pad=(ph, pw), alpha=alpha)
        assert rel(dfilt.cpu().numpy().reshape(rdf.shape), rdf) <= TOL[kernel], ("wgrad", shape)
        try:
            need = mx.conv2_bprop_data_workspace(d, KIND[kernel])
            ws = torch.empty(max(16, need), dtype=torch.uint8, device="cuda")
            din = torch.full((inp.size,), float("nan"), device="cuda")
            mx.conv2_bprop_data(d, g, f, din, ws, KIND[kernel])
        except mx.MaxdnnError as e:
            assert e.status == mx.NOT_SUPPORTED, ("dgrad", shape)    # transposed problem refused
        else:
            rdi = oracle.conv2_bprop_data(rg, rf, (Hi, Wi), stride=(sh, sw), pad=(ph, pw), alpha=alpha)
            assert rel(din.cpu().numpy().reshape(rdi.shape), rdi) <= TOL[kernel], ("dgrad", shape)
        done += 1
    assert mx.last_device_status() == mx.OK


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
def test_random_few_channel_strided_shapes(kernel):
    """Few channels, stride > 1, large filters: the plan that merges filter columns into K
    and stages one patch strip per step (or one box per pixel where the window shift is not
    a whole swizzle group), with one or several filter rows per step as the stage budget
    decides; wide maps so that tiles hold several pixels and the last tile of a row is
    ragged."""
    rng = np.random.default_rng({"tf32": 44, "bf16": 55}[kernel])
    atom = {"tf32": 32, "bf16": 64}[kernel]
    done = 0
    while done < 40:
        Sk = int(rng.integers(2, 12))
        stride = int(rng.integers(2, 5))
        pad = int(rng.integers(0, min(Sk, 4)))
        Wi = int(rng.integers(Sk, 64))
        Hi = int(rng.integers(Sk, 20))
        Nb = atom * int(rng.integers(1, 3))
        Nc = int(rng.integers(1, 8 if kernel == "tf32" else 16))
        No = 32 * int(rng.integers(1, 6))
        alpha = float(rng.choice([1.0, -0.5]))
        w = wl.Workload("fuzz_fc", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", -1.0, 1.0),
                        ("uniform", -1.0, 1.0), 9500 + done)
        d = mx.ConvDesc.make(*w.dims)
        inp, filt = wl.make_inputs(w)
        (x, f), (rx, rf) = operands(kernel, inp, filt)
        out = torch.full((mx.conv_out_elems(d),), float("nan"), device="cuda")
        st = mx.fprop_status(d, x, f, out, KIND[kernel])
        if st == mx.NOT_SUPPORTED:
            continue                      # a step of this shape does not fit two ring stages
        assert st == mx.OK, w.dims
        assert mx.last_device_status() == mx.OK
        ref = oracle.conv_fprop(rx, rf, stride=stride, pad=pad, alpha=alpha)
        assert rel(out.cpu().numpy().reshape(ref.shape), ref) <= TOL[kernel], w.dims
        done += 1


def test_random_shapes_three_product_tf32():
    """maxdnn_conv_fprop_tf32x3 (chunked accumulation) on random shapes, held to the exact
    kernel's bar: ragged tiles, dead column groups, one chunk or many, all plans."""
    done = 0
    for i, shape in enumerate(random_shapes("tf32", 40, 66)):
        Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
        w = wl.Workload("fuzz_x3", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", -1.0, 1.0),
                        ("uniform", -1.0, 1.0), 9700 + i)
        inp, filt = wl.make_inputs(w)
        d = mx.ConvDesc.make(*w.dims)
        ws = torch.empty(max(16, mx.conv_fprop_tf32x3_workspace(d)), dtype=torch.uint8, device="cuda")
        out = torch.full((mx.conv_out_elems(d),), float("nan"), device="cuda")
        try:
            mx.conv_fprop_tf32x3(d, torch.from_numpy(inp).cuda(), torch.from_numpy(filt).cuda(), out, ws)
        except mx.MaxdnnError as e:
            assert e.status == mx.NOT_SUPPORTED      # 3 Nc channels x Sk^2 taps: too many K steps
            continue
        assert mx.last_device_status() == mx.OK, shape
        ref = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
        assert rel(out.cpu().numpy().reshape(ref.shape), ref) <= 1e-5, shape
        done += 1
    assert done >= 30
