"""Parity of the backward-propagation entry points against the CPU oracle, through the
C ABI: the gradient with respect to the maps (an FPROP of the output gradient with the
transformed filter bank, on all three kernels) and with respect to the filters (exact
fp32, split reduction with a fixed-order sum)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu

KIND = {"fp32": mx.KERNEL_FP32, "tf32": mx.KERNEL_TF32, "bf16": mx.KERNEL_BF16}
TOL = {"fp32": 1e-5, "tf32": 5e-3, "bf16": 2e-2}


def make(shape, seed):
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    w = wl.Workload("bprop", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), seed)
    inp, filt = wl.make_inputs(w)
    return w, inp, filt, wl.make_dout(w)


def rel_err(got, ref):
    return float(np.max(np.abs(got.astype(np.float64) - ref))) / max(float(np.max(np.abs(ref))), 1e-30)


def dev(a, kernel):
    if kernel == "bf16":
        return torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def rounded(a, kernel):
    """What the kernel's operands really are: bf16 operands are the caller's rounding."""
    return wl.from_bf16_bits(wl.to_bf16_bits(a)) if kernel == "bf16" else a


DGRAD_SHAPES = [
    # Nb Wi Hi Nc No Sk stride pad alpha
    (64, 14, 9, 64, 96, 3, 1, 1, 1.0),
    (128, 9, 7, 32, 64, 5, 1, 2, 0.5),
    (64, 12, 10, 128, 32, 3, 1, 0, 1.0),      # no padding: din gets pad' = Sk - 1
    (64, 8, 8, 64, 64, 1, 1, 0, 2.0),         # 1x1
    (64, 10, 6, 96, 160, 4, 1, 3, 1.0),       # even filter, pad = Sk - 1
]


@pytest.mark.parametrize("kernel", ["fp32", "tf32", "bf16"])
@pytest.mark.parametrize("shape", DGRAD_SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_data(kernel, shape):
    w, inp, filt, dout = make(shape, 900 + shape[5])
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_workspace(d, KIND[kernel]), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data(d, dev(dout, kernel), dev(filt, kernel), din, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_data(rounded(dout, kernel), rounded(filt, kernel), (w.Hi, w.Wi),
                                 stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = din.cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    assert rel_err(got, ref) <= TOL[kernel]


DGRAD_STRIDED_SHAPES = [
    # Nb Wi Hi Nc No Sk stride pad alpha
    (64, 15, 11, 32, 64, 3, 2, 1, 1.0),       # classes with 2x2, 2x1, 1x2, 1x1 taps
    (64, 16, 12, 32, 32, 2, 2, 0, 0.5),       # filter = stride: one tap per class
    (64, 35, 27, 8, 32, 11, 4, 0, 1.0),       # the first-layer geometry: 16 classes, 3x3 / 3x2 / 2x2 taps
    (64, 23, 19, 4, 32, 11, 4, 2, 1.0),       # with padding: classes start at different rows
    (64, 23, 19, 32, 64, 7, 4, 3, 1.0),       # the same with 32 channels (tensor kernels too)
    (64, 14, 14, 32, 32, 2, 3, 0, 1.0),       # stride > filter: a class without taps stays zero
    (64, 13, 10, 32, 32, 3, 2, 2, 1.0),       # pad = Sk - 1: a class whose window skips a row of dout
    (64, 9, 9, 32, 32, 5, 3, 1, -1.0),
]


@pytest.mark.parametrize("kernel", ["fp32", "tf32", "bf16"])
@pytest.mark.parametrize("shape", DGRAD_STRIDED_SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_data_strided(kernel, shape):
    """Stride > 1: one FPROP per residue class of the map positions, scattered onto its grid."""
    if kernel != "fp32" and shape[3] % 32:
        pytest.skip("the tensor-core kernels want a multiple of 32 'filters' (here: channels)")
    w, inp, filt, dout = make(shape, 1300 + shape[5])
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_workspace(d, KIND[kernel]), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data(d, dev(dout, kernel), dev(filt, kernel), din, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_data(rounded(dout, kernel), rounded(filt, kernel), (w.Hi, w.Wi),
                                 stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = din.cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    assert rel_err(got, ref) <= TOL[kernel]


def test_bprop_data_refusals():
    d = mx.ConvDesc.make(64, 16, 16, 32, 32, 3, 1, 3, 1.0)          # pad > Sk - 1, stride 1
    with pytest.raises(mx.MaxdnnError) as e:
        mx.conv_bprop_data_workspace(d)
    assert e.value.status == mx.NOT_SUPPORTED
    d = mx.ConvDesc.make(64, 16, 16, 32, 32, 3, 1, 1, 1.0)
    need = mx.conv_bprop_data_workspace(d)
    assert need == 32 * 9 * 32 * 4
    g = torch.zeros(mx.conv_out_elems(d), device="cuda")
    f = torch.zeros(mx.conv_filt_elems(d), device="cuda")
    x = torch.zeros(mx.conv_in_elems(d), device="cuda")
    small = torch.empty(need - 16, dtype=torch.uint8, device="cuda")
    assert mx.bprop_data_status(d, g, f, x, small) == mx.INVALID_VALUE


WGRAD_SHAPES = [
    # Nb Wi Hi Nc No Sk stride pad alpha
    (64, 14, 9, 20, 96, 3, 1, 1, 1.0),        # 14 channels per tile: two channel blocks
    (128, 9, 7, 12, 64, 5, 1, 2, 0.5),        # 5 channels per tile, ragged last block
    (32, 23, 19, 3, 96, 11, 4, 0, 1.0),       # the first-layer shape: all 121 taps x 1 channel
    (36, 12, 10, 16, 132, 3, 2, 1, 1.0),      # images and filters not multiples of 32 / 128
    (64, 8, 8, 160, 64, 1, 1, 0, 2.0),        # 1x1: 128 channels per tile
    (8, 30, 30, 4, 8, 13, 1, 6, 1.0),         # 13x13 filter: 9 filter rows per tile, two row blocks
    (64, 10, 6, 8, 256, 4, 1, 3, -1.0),       # two filter blocks
]


@pytest.mark.parametrize("splits", [0, 1, 3])
@pytest.mark.parametrize("shape", WGRAD_SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_filter(shape, splits, monkeypatch):
    if splits:
        mx.set_option("WGRAD_SPLITS", splits)
    w, inp, filt, dout = make(shape, 1700 + shape[5])
    d = mx.ConvDesc.make(*w.dims)
    need = mx.conv_bprop_filter_workspace(d)
    if splits == 1:
        assert need == 0
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda") if need else None
    dfilt = torch.full((mx.conv_filt_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_filter(d, torch.from_numpy(inp).cuda(), torch.from_numpy(dout).cuda(), dfilt, ws)
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_filter(inp, dout, w.Sk, stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = dfilt.cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    assert rel_err(got, ref) <= 1e-5


WGRAD_TC_SHAPES = WGRAD_SHAPES + [
    (64, 14, 9, 40, 96, 3, 1, 1, 1.0),        # 28 channels x 9 taps = 252 rows per tile, two blocks
    (128, 9, 7, 24, 64, 5, 1, 2, 0.5),        # 10 channels x 25 taps
    (64, 8, 8, 300, 64, 1, 1, 0, 2.0),        # 1x1: 256 channels per tile, ragged second block
]


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
@pytest.mark.parametrize("pair", [-1, 1])
@pytest.mark.parametrize("splits", [0, 2])
@pytest.mark.parametrize("shape", WGRAD_TC_SHAPES + [(64, 9, 9, 64, 512, 3, 1, 1, 1.0),
                                                     (64, 9, 9, 33, 384, 3, 1, 1, 1.0)],
                         ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_filter_tensor_cores(shape, splits, pair, kernel, monkeypatch):
    """pair = -1: one-SM tiles of 128 filters; 1: two-SM tiles of 256 filters (each CTA stages
    its 128 filters and half of the tile's channels), forced also where the planner would not
    take them (fewer than 129 filters: the second CTA's filters are all out of range)."""
    if kernel == "bf16" and shape[0] % 8:
        pytest.skip("a row of bf16 images must be a multiple of 16 bytes")
    if pair == 1 and shape[3] == 3 and shape[5] == 11:
        pytest.skip("one channel per tile (121 taps): nothing to split between two CTAs")
    mx.set_option("WGRAD_PAIR", pair)
    if splits:
        mx.set_option("WGRAD_SPLITS", splits)
    w, inp, filt, dout = make(shape, 2600 + shape[5])
    d = mx.ConvDesc.make(*w.dims)
    need = mx.conv_bprop_filter_workspace(d, KIND[kernel])
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda") if need else None
    dfilt = torch.full((mx.conv_filt_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_filter(d, dev(inp, kernel), dev(dout, kernel), dfilt, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_filter(rounded(inp, kernel), rounded(dout, kernel), w.Sk,
                                   stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = dfilt.cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    assert rel_err(got, ref) <= TOL[kernel]


def test_bprop_filter_is_reproducible():
    """Partial sums are added in a fixed order: two runs agree bit for bit."""
    w, inp, filt, dout = make((64, 14, 9, 20, 96, 3, 1, 1, 1.0), 77)
    d = mx.ConvDesc.make(*w.dims)
    need = mx.conv_bprop_filter_workspace(d)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    a = torch.empty(mx.conv_filt_elems(d), device="cuda")
    b = torch.empty_like(a)
    x, g = torch.from_numpy(inp).cuda(), torch.from_numpy(dout).cuda()
    mx.conv_bprop_filter(d, x, g, a, ws)
    mx.conv_bprop_filter(d, x, g, b, ws)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


@pytest.mark.parametrize("name,kernel", [("first11x11s4", "fp32"), ("mid5x5", "fp32"), ("wide3x3", "fp32"),
                                         ("mid5x5", "tf32"), ("large3x3", "bf16"), ("first11x11s4", "bf16")])
def test_full_size_sampled_bprop_filter(name, kernel):
    """Benchmark sizes, in the launch configuration the bench times: random single
    gradient elements against the oracle (fp32: within the a-priori bound of an fp32 sum)."""
    w = wl.WORKLOADS[name]
    inp, _ = wl.make_inputs(w)
    dout = wl.make_dout(w)
    d = mx.ConvDesc.make(*w.dims)
    need = mx.conv_bprop_filter_workspace(d, KIND[kernel])
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    dfilt = torch.full((mx.conv_filt_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_filter(d, dev(inp, kernel), dev(dout, kernel), dfilt, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    got = dfilt.cpu().numpy().reshape(w.Nc, w.Sk, w.Sk, w.No)
    assert np.isfinite(got).all()
    r_in, r_g = rounded(inp, kernel), rounded(dout, kernel)
    R = dout.shape[1] * dout.shape[2] * w.Nb
    rng = np.random.default_rng(4)
    pts = [tuple(int(rng.integers(0, s)) for s in got.shape) for _ in range(200)]
    vals = [oracle.conv_bprop_filter_point(r_in, r_g, w.Sk, *p, stride=w.stride, pad=w.pad,
                                           alpha=w.alpha) for p in pts]
    scale = max(abs(v) for v, _ in vals)
    for p, (v, a) in zip(pts, vals):
        if kernel == "tf32":
            assert abs(float(got[p]) - v) <= TOL[kernel] * scale
        else:
            # fp32 products and sums (bf16 operands multiply exactly in fp32); partial sums in
            # blocks: the plain bound R u |terms| is loose, 64 sqrt(R) u |terms| holds with margin
            assert abs(float(got[p]) - v) <= 64 * np.sqrt(R) * 2.0 ** -24 * abs(w.alpha) * a + 1e-30


@pytest.mark.parametrize("name,kernel", [("mid5x5", "fp32"), ("large3x3", "bf16"), ("wide3x3", "tf32")])
def test_full_size_sampled_bprop_data(name, kernel):
    w = wl.WORKLOADS[name]
    _, filt = wl.make_inputs(w)
    dout = wl.make_dout(w)
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_workspace(d, KIND[kernel]), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data(d, dev(dout, kernel), dev(filt, kernel), din, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    got = din.cpu().numpy().reshape(w.Nc, w.Hi, w.Wi, w.Nb)
    assert np.isfinite(got).all()
    rd, rf = rounded(dout, kernel), rounded(filt, kernel)
    rng = np.random.default_rng(5)
    pts = [tuple(int(rng.integers(0, s)) for s in got.shape) for _ in range(200)]
    pts += [(0, 0, 0, 0), (w.Nc - 1, w.Hi - 1, w.Wi - 1, w.Nb - 1), (1, 0, w.Wi - 1, 3)]   # corners: apron
    vals = [oracle.conv_bprop_data_point(rd, rf, (w.Hi, w.Wi), *p, stride=w.stride, pad=w.pad,
                                         alpha=w.alpha) for p in pts]
    scale = max(abs(v) for v, _ in vals)
    K = w.No * w.Sk ** 2
    for p, (v, a) in zip(pts, vals):
        if kernel == "fp32":
            assert abs(float(got[p]) - v) <= (K + 3) * 2.0 ** -24 * abs(w.alpha) * a + 1e-30
        else:
            assert abs(float(got[p]) - v) <= TOL[kernel] * scale


@pytest.mark.parametrize("kernel", ["fp32", "bf16"])
def test_full_size_sampled_strided_bprop_data(kernel):
    """A full-size stride-2 layer (56 x 56 x 128 -> 256, 3 x 3): four classes with 2x2, 2x1, 1x2
    and 1x1 taps; sampled elements of din, corners and both parities of h, w included."""
    w = wl.WORKLOADS["large3x3"].scaled(stride=2)
    _, filt = wl.make_inputs(w)
    dout = wl.make_dout(w)
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_workspace(d, KIND[kernel]), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data(d, dev(dout, kernel), dev(filt, kernel), din, ws, KIND[kernel])
    assert mx.last_device_status() == mx.OK
    got = din.cpu().numpy().reshape(w.Nc, w.Hi, w.Wi, w.Nb)
    assert np.isfinite(got).all()
    rd, rf = rounded(dout, kernel), rounded(filt, kernel)
    rng = np.random.default_rng(6)
    pts = [tuple(int(rng.integers(0, s)) for s in got.shape) for _ in range(200)]
    pts += [(0, 0, 0, 0), (0, 0, 1, 0), (0, 1, 0, 0), (0, 1, 1, 0),
            (w.Nc - 1, w.Hi - 1, w.Wi - 1, w.Nb - 1), (5, w.Hi - 2, w.Wi - 1, 7)]
    vals = [oracle.conv_bprop_data_point(rd, rf, (w.Hi, w.Wi), *p, stride=w.stride, pad=w.pad,
                                         alpha=w.alpha) for p in pts]
    scale = max(abs(v) for v, _ in vals)
    for p, (v, a) in zip(pts, vals):
        assert abs(float(got[p]) - v) <= 1e-5 * scale, p


@pytest.mark.parametrize("kind", [mx.KERNEL_FP32, mx.KERNEL_TF32, mx.KERNEL_BF16, "tf32x3"])
def test_unsupported_strided_map_gradient_launches_nothing(kind):
    """A strided map gradient whose per-class sub-problems have no plan (their 'filters' are
    the layer's channels: 3 here, against the 16-byte row rule) is refused before anything
    is enqueued: no memset, no split, no transform kernel."""
    d = mx.ConvDesc.make(64, 23, 23, 3, 32, 5, 2, 1)
    Ho, Wo = mx.conv_out_dims(d)
    bf16 = kind == mx.KERNEL_BF16
    dt = torch.bfloat16 if bf16 else torch.float32
    dout = torch.zeros(32 * Ho * Wo * 64, dtype=dt, device="cuda")
    filt = torch.zeros(mx.conv_filt_elems(d), dtype=dt, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), 7.0, dtype=torch.float32, device="cuda")
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    before = mx.launch_count()
    with pytest.raises(mx.MaxdnnError) as e:
        if kind == "tf32x3":
            mx.conv_bprop_data_tf32x3(d, dout, filt, din, ws)
        else:
            mx.conv_bprop_data(d, dout, filt, din, ws, kind)
    assert e.value.status == mx.NOT_SUPPORTED
    assert mx.launch_count() == before
    torch.cuda.synchronize()
    assert bool((din == 7.0).all())           # not cleared, not written
