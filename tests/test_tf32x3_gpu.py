"""Three-product TF32 FPROP (fp32 operands split into hi + lo, one TF32 launch over 3 Nc
channels, the sum over K accumulated in chunks that are added in round-to-nearest fp32):
required here is the exact kernel's own bar, <= 1e-5 of the largest output against the fp64
oracle, whatever the length K of the sums (measured 1e-6 .. 3e-6).  Without the chunks
(MAXDNN_X3_CHUNK_ROWS=0) the tensor core's truncating accumulator costs about 1e-8 K on
same-signed data; that path is kept as a switch and held to max(5e-5, 1.2e-8 K)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu
TOL_X3 = 1e-5


def run(w, inp, filt):
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_fprop_tf32x3_workspace(d), dtype=torch.uint8, device="cuda")
    out = torch.full((mx.conv_out_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_fprop_tf32x3(d, torch.from_numpy(inp).cuda(), torch.from_numpy(filt).cuda(), out, ws)
    assert mx.last_device_status() == mx.OK
    Ho, Wo = mx.conv_out_dims(d)
    return out.cpu().numpy().reshape(w.No, Ho, Wo, w.Nb)


@pytest.mark.parametrize("shape", [
    (64, 14, 9, 32, 64, 3, 1, 1, 1.0),
    (128, 9, 7, 48, 96, 5, 1, 2, 0.5),
    (32, 23, 19, 3, 96, 11, 4, 0, 1.0),      # 9 split channels: filter columns merged into K
    (64, 12, 10, 100, 256, 3, 2, 1, 1.0),
], ids=lambda s: "x".join(str(v) for v in s))
def test_tf32x3_small(shape):
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    w = wl.Workload("x3", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 4400 + Sk)
    inp, filt = wl.make_inputs(w)
    got = run(w, inp, filt)
    ref = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    assert np.isfinite(got).all()
    err = float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref)))
    assert err <= TOL_X3
    # and it really is better than one TF32 product: the plain TF32 kernel on the same data
    d = mx.ConvDesc.make(*w.dims)
    out1 = torch.empty(mx.conv_out_elems(d), device="cuda")
    mx.conv_fprop_tf32(d, torch.from_numpy(inp).cuda(), torch.from_numpy(filt).cuda(), out1)
    err1 = float(np.max(np.abs(out1.cpu().numpy().reshape(ref.shape).astype(np.float64) - ref))) / \
        float(np.max(np.abs(ref)))
    assert err < err1 / 8


@pytest.mark.parametrize("pair", [1, -1])
@pytest.mark.parametrize("shape", [
    (64, 14, 9, 48, 256, 3, 1, 1, 1.0),       # strip reuse, two tiles of 256 filters
    (128, 9, 7, 32, 256, 5, 1, 2, 1.0),       # the CTAs of a pair split the images
    (32, 21, 5, 40, 256, 3, 1, 1, 1.0),       # 8 pixels x 32 images, split by pixel
    (64, 13, 5, 24, 512, 3, 1, 1, 0.5),       # ragged pixel tail
    (64, 12, 6, 24, 160, 3, 1, 1, 1.0),       # 160 filters: second CTA of the pair mostly idle
    (64, 9, 9, 300, 256, 3, 1, 1, 1.0),       # K = 2700: several chunks per tile
], ids=lambda s: "x".join(str(v) for v in s))
def test_tf32x3_both_chunked_kernels(shape, pair, monkeypatch):
    """The chunked kernel on one-SM tiles (pair = -1) and on two-SM tiles (pair = 1, forced
    also where the planner would not take them), against the oracle at the exact kernel's bar."""
    mx.set_option("UMMA_PAIR", pair)
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    w = wl.Workload("x3p", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", 0.0, 1.0),
                    ("uniform", 0.0, 1.0), 4500 + Nc)          # same-signed terms: the hard case
    inp, filt = wl.make_inputs(w)
    d = mx.ConvDesc.make(Nb, Wi, Hi, 3 * Nc, No, Sk, stride, pad, alpha)
    assert mx.conv_plan_query(d, mx.KERNEL_TF32, 148)[0].tile_m == (256 if pair == 1 else 128)
    got = run(w, inp, filt)
    ref = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    assert np.isfinite(got).all()
    assert float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref))) <= TOL_X3


@pytest.mark.parametrize("chunked", [True, False])
@pytest.mark.parametrize("name", ["mid5x5", "wide3x3", "large3x3", "first11x11s4", "alexnet_conv2",
                                  "overfeat_L3", "overfeat_L5"])
def test_tf32x3_full_size_sampled(name, chunked, monkeypatch):
    w = wl.ALL[name]
    tol = TOL_X3
    if not chunked:
        if name not in ("mid5x5", "overfeat_L5"):
            pytest.skip("one-accumulator path: two layers are enough")
        mx.set_option("X3_CHUNK_ROWS", 0)
        tol = max(5e-5, 1.2e-8 * w.Nc * w.Sk * w.Sk)      # overfeat_L5: K = 9216
    inp, filt = wl.make_inputs(w)
    got = run(w, inp, filt)
    assert np.isfinite(got).all()
    Ho = got.shape[1]
    for y in sorted({0, Ho // 2, Ho - 1}):
        ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha,
                                rows=(y, y + 1))[:, y]
        err = float(np.max(np.abs(got[:, y].astype(np.float64) - ref))) / float(np.max(np.abs(ref)))
        assert err <= tol


@pytest.mark.parametrize("shape", [
    (64, 14, 9, 64, 96, 3, 1, 1, 1.0),        # transposed problem: 96 channels -> 64 "filters"
    (128, 9, 7, 96, 64, 5, 1, 2, 0.5),
    (64, 12, 10, 128, 32, 3, 1, 0, 1.0),      # no padding: the gradient's FPROP pads by Sk - 1
    (32, 16, 16, 256, 160, 3, 1, 1, -2.0),    # two-SM tiles (256 "filters"), K = 1440
], ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_data_tf32x3(shape):
    """Map gradient in the three-product mode against the gradient oracle, at the exact
    kernel's bar (same-signed operands: the case the chunked accumulation is for)."""
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    w = wl.Workload("x3g", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", 0.0, 1.0),
                    ("uniform", 0.0, 1.0), 4600 + Nc)
    _, filt = wl.make_inputs(w)
    dout = np.abs(wl.make_dout(w))
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_tf32x3_workspace(d), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data_tf32x3(d, torch.from_numpy(dout).cuda(), torch.from_numpy(filt).cuda(), din, ws)
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    got = din.cpu().numpy().reshape(ref.shape)
    assert np.isfinite(got).all()
    assert float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref))) <= TOL_X3


def test_bprop_data_tf32x3_full_size_sampled_and_refusals():
    w = wl.WORKLOADS["large3x3"]
    _, filt = wl.make_inputs(w)
    dout = wl.make_dout(w)
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_tf32x3_workspace(d), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data_tf32x3(d, torch.from_numpy(dout).cuda(), torch.from_numpy(filt).cuda(), din, ws)
    assert mx.last_device_status() == mx.OK
    got = din.cpu().numpy().reshape(w.Nc, w.Hi, w.Wi, w.Nb)
    assert np.isfinite(got).all()
    rng = np.random.default_rng(12)
    pts = [tuple(int(rng.integers(0, s)) for s in got.shape) for _ in range(150)]
    pts += [(0, 0, 0, 0), (w.Nc - 1, w.Hi - 1, w.Wi - 1, w.Nb - 1)]
    vals = [oracle.conv_bprop_data_point(dout, filt, (w.Hi, w.Wi), *p, stride=1, pad=w.pad,
                                         alpha=w.alpha)[0] for p in pts]
    scale = max(abs(v) for v in vals)
    assert max(abs(float(got[p]) - v) for p, v in zip(pts, vals)) <= TOL_X3 * scale
    with pytest.raises(mx.MaxdnnError) as e:        # pad > Sk - 1 at stride 1: no transposed FPROP
        mx.conv_bprop_data_tf32x3_workspace(mx.ConvDesc.make(64, 16, 16, 32, 32, 3, 1, 3, 1.0))
    assert e.value.status == mx.NOT_SUPPORTED


@pytest.mark.parametrize("shape", [
    (64, 15, 11, 32, 64, 3, 2, 1, 1.0),       # classes with 2x2, 2x1, 1x2, 1x1 taps
    (64, 16, 12, 32, 32, 2, 2, 0, 0.5),       # filter = stride: one tap per class
    (64, 23, 19, 32, 64, 7, 4, 3, 1.0),       # stride 4: sixteen classes
    (64, 14, 14, 32, 32, 2, 3, 0, 1.0),       # stride > filter: a class without taps stays zero
    (32, 13, 10, 64, 96, 3, 2, 2, -1.0),      # pad = Sk - 1: a class whose window skips a row of dout
], ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_data_tf32x3_strided(shape):
    """Stride > 1: every residue class through the chunked kernels (the gradient split once,
    each class's sub-filter bank split after its transform), at the exact kernel's bar."""
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    w = wl.Workload("x3s", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", 0.0, 1.0),
                    ("uniform", 0.0, 1.0), 4800 + Sk)
    _, filt = wl.make_inputs(w)
    dout = np.abs(wl.make_dout(w))
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_data_tf32x3_workspace(d), dtype=torch.uint8, device="cuda")
    din = torch.full((mx.conv_in_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_data_tf32x3(d, torch.from_numpy(dout).cuda(), torch.from_numpy(filt).cuda(), din, ws)
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    got = din.cpu().numpy().reshape(ref.shape)
    assert np.isfinite(got).all()
    assert float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref))) <= TOL_X3


@pytest.mark.parametrize("pair", [-1, 1])
@pytest.mark.parametrize("splits", [0, 1, 3])
@pytest.mark.parametrize("shape", [
    (64, 14, 9, 40, 96, 3, 1, 1, 1.0),        # 28 channels x 9 taps per tile, two channel blocks
    (128, 9, 7, 24, 64, 5, 1, 2, 0.5),        # 10 channels x 25 taps
    (32, 23, 19, 3, 96, 11, 4, 0, 1.0),       # the first-layer shape: two blocks of filter rows
    (64, 8, 8, 300, 64, 1, 1, 0, 2.0),        # 1x1: 256 channels per tile, ragged second block
    (64, 12, 10, 16, 132, 3, 2, 1, 1.0),      # filters not a multiple of 128, stride 2
    (96, 10, 6, 8, 256, 4, 1, 3, -1.0),       # two filter blocks; 96 images = three 128-byte rows
], ids=lambda s: "x".join(str(v) for v in s))
def test_bprop_filter_tf32x3(shape, splits, pair, monkeypatch):
    """Filter gradient in the three-product mode (the three products as one reduction over
    three times the images, accumulated in chunks) against the gradient oracle at the exact
    kernel's bar; same-signed operands, forced split counts, one-SM (pair = -1) and two-SM
    tiles (pair = 1, forced also where the planner would not take them)."""
    mx.set_option("WGRAD_PAIR", pair)
    if splits:
        mx.set_option("WGRAD_SPLITS", splits)
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    w = wl.Workload("x3w", Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha, ("uniform", 0.0, 1.0),
                    ("uniform", 0.0, 1.0), 4700 + Nc)
    inp, _ = wl.make_inputs(w)
    dout = np.abs(wl.make_dout(w))
    d = mx.ConvDesc.make(*w.dims)
    ws = torch.empty(mx.conv_bprop_filter_tf32x3_workspace(d), dtype=torch.uint8, device="cuda")
    dfilt = torch.full((mx.conv_filt_elems(d),), float("nan"), dtype=torch.float32, device="cuda")
    mx.conv_bprop_filter_tf32x3(d, torch.from_numpy(inp).cuda(), torch.from_numpy(dout).cuda(), dfilt, ws)
    assert mx.last_device_status() == mx.OK
    ref = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    got = dfilt.cpu().numpy().reshape(ref.shape)
    assert np.isfinite(got).all()
    assert float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref))) <= TOL_X3
