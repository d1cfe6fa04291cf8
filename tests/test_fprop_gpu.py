"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs, element by element."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5   # max |gpu - oracle| / max |oracle|


def run_fp32(w, inp, filt, canary=True):
    """Run the fp32 kernel; the output buffer sits between two canary strips."""
    d = mx.ConvDesc.make(*w.dims)
    n_out = mx.conv_out_elems(d)
    guard = 1024
    buf = torch.full((n_out + 2 * guard,), 12345.0, dtype=torch.float32, device="cuda")
    out = buf[guard:guard + n_out]
    d_in = torch.from_numpy(inp).cuda()
    d_f = torch.from_numpy(filt).cuda()
    mx.conv_fprop(d, d_in, d_f, out)
    assert mx.last_device_status() == mx.OK
    host = buf.cpu().numpy()
    if canary:
        assert np.all(host[:guard] == 12345.0) and np.all(host[guard + n_out:] == 12345.0)
    Ho, Wo = mx.conv_out_dims(d)
    return host[guard:guard + n_out].reshape(w.No, Ho, Wo, w.Nb)


def rel_inf(g, r):
    return float(np.max(np.abs(g.astype(np.float64) - r.astype(np.float64)))) / \
        max(float(np.max(np.abs(r))), 1e-30)


def check_fp32(w, inp=None, filt=None):
    if inp is None:
        inp, filt = wl.make_inputs(w)
    ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha)
    got = run_fp32(w, inp, filt)
    assert got.shape == ref.shape
    err = rel_inf(got, ref)
    assert err <= TOL_FP32, "E_inf = %.3e" % err
    # a-priori bound of an fp32 dot product of K terms, per element:
    # |gpu - exact| <= (K + 3) 2^-24 |alpha| sum |f x|  (+ the oracle's own rounding)
    K = w.Nc * w.Sk * w.Sk
    abs_sum = oracle.conv_fprop(np.abs(inp), np.abs(filt), stride=w.stride, pad=w.pad,
                                alpha=abs(w.alpha)).astype(np.float64)
    bound = (K + 3) * 2.0 ** -24 * abs_sum * (1 + 2.0 ** -20) + 1e-37
    assert np.all(np.abs(got.astype(np.float64) - ref.astype(np.float64)) <= bound)
    return got


def test_tiny_workload_fp32():
    check_fp32(wl.WORKLOADS["tiny3x3"])


@pytest.mark.parametrize("name,kw", [
    # reduced copies of the benchmark layers: several tiles, ragged tails
    ("first11x11s4", dict(Nb=128, Wi=51, Hi=43, No=96)),
    ("first11x11s4", dict(Nb=32, Wi=39, Hi=39, No=96)),
    ("mid5x5", dict(Nb=128, Wi=9, Hi=7, Nc=96, No=256)),
    ("mid5x5", dict(Nb=64, Wi=11, Hi=11, Nc=40, No=160)),
    ("wide3x3", dict(Nb=128, Wi=6, Hi=5, Nc=256, No=384)),
    ("large3x3", dict(Nb=64, Wi=14, Hi=9, Nc=128, No=256)),
])
def test_scaled_workloads_fp32(name, kw):
    check_fp32(wl.WORKLOADS[name].scaled(**kw))


EDGE = [
    # Nb  Wi  Hi  Nc  No  Sk st pad alpha
    (4, 5, 5, 1, 4, 1, 1, 0, 1.0),          # smallest legal sizes, 1x1 filter
    (4, 7, 6, 3, 4, 3, 1, 1, -2.0),         # few channels: whole filter rows per K step
    (8, 9, 9, 2, 12, 5, 2, 2, 1.0),         # stride 2 with padding
    (132, 6, 5, 9, 100, 3, 1, 1, 0.5),      # ragged image chunk and ragged filter block
    (36, 10, 7, 17, 36, 3, 3, 1, 1.0),      # stride 3, channel tail in the last K step
    (20, 13, 4, 33, 68, 2, 1, 0, 1.0),      # even filter, Wi != Hi, odd tiles
    (64, 5, 5, 8, 32, 5, 1, 0, 1.0),        # single output pixel
    (32, 8, 8, 16, 32, 3, 1, 3, 1.0),       # pad as large as the filter: all-apron patches
    (256, 4, 4, 12, 32, 3, 1, 1, 0.0),      # alpha = 0, two image chunks
    (16, 30, 3, 5, 8, 3, 1, 1, 1.0),        # wide short map, many pixels per tile
]


@pytest.mark.parametrize("shape", EDGE, ids=lambda s: "x".join(str(v) for v in s))
def test_edge_shapes_fp32(shape):
    Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha = shape
    w = wl.Workload("edge", Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 4242 + Nb + No)
    check_fp32(w)


@pytest.mark.parametrize("tile_m,cols", [(32, 128), (64, 128), (96, 128), (128, 128), (256, 128), (64, 256),
                                         (96, 256), (128, 256)])
@pytest.mark.parametrize("stride", [1, 2])
def test_every_tile_shape(tile_m, cols, stride, monkeypatch):
    """Every kernel instance (register block, producer placement, one box per stage
    or one per pixel) on a shape with ragged filter, image and pixel tails."""
    mx.set_option("FFMA_TILE_M", tile_m)
    mx.set_option("FFMA_COLS", cols)
    w = wl.Workload("tiles", 64, 11, 8, 24, 296, 3, stride, 1, 1.0, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 99)
    d = mx.ConvDesc.make(*w.dims)
    info, _ = mx.conv_plan_query(d, mx.KERNEL_FP32, 148)
    assert info.tile_m == tile_m and info.tile_px * info.tile_n <= cols
    check_fp32(w)


SPLIT = [
    # shapes whose plan splits the last wave of tiles along K (more tiles than CTAs, a
    # partly filled last wave), with the tile shape pinned so that every register block's
    # partial-sum path runs: (dims, tile_m, cols)
    ((128, 15, 13, 32, 128, 3, 1, 1, 1.0), 0, 0),
    ((64, 24, 17, 24, 256, 3, 1, 1, 0.5), 0, 0),
    ((128, 14, 12, 40, 200, 5, 1, 2, 1.0), 0, 0),
    ((128, 16, 10, 128, 128, 3, 1, 1, 1.0), 0, 0),
    ((128, 16, 10, 24, 96, 3, 1, 1, 1.0), 32, 128),
    ((128, 16, 12, 24, 192, 3, 1, 1, 1.0), 96, 128),
    ((128, 20, 18, 24, 256, 3, 1, 1, 1.0), 256, 128),
    ((64, 40, 18, 40, 128, 3, 1, 1, 1.0), 128, 256),
    ((64, 80, 36, 40, 64, 3, 2, 1, 1.0), 64, 256),
    ((64, 40, 18, 40, 64, 3, 1, 1, 1.0), 64, 256),
    ((64, 40, 36, 16, 96, 3, 1, 1, 1.0), 96, 256),
    ((128, 55, 83, 3, 96, 11, 4, 0, 1.0), 96, 128),      # 11 filter rows in steps of 2: a short last step
    ((128, 13, 9, 96, 256, 3, 1, 1, 1.0), 128, 128),     # 96 channels per step: the long-iteration instance
]


@pytest.mark.parametrize("dims,tile_m,cols", SPLIT, ids=lambda v: "x".join(str(x) for x in v)
                         if isinstance(v, tuple) else str(v))
def test_split_tail_fp32(dims, tile_m, cols):
    """The tail wave split along K: contributions through the workspace, finishers adding
    them in CTA order — against the oracle, and bitwise equal from run to run."""
    mx.set_option("FFMA_STREAMK", 2)       # split whenever there is a tail, whatever its length
    if tile_m:
        mx.set_option("FFMA_TILE_M", tile_m)
        mx.set_option("FFMA_COLS", cols)
    w = wl.Workload("split", *dims, ("uniform", -1.0, 1.0), ("uniform", -1.0, 1.0), 321)
    d = mx.ConvDesc.make(*w.dims)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    info, _ = mx.conv_plan_query(d, mx.KERNEL_FP32, sms)
    assert info.split_tiles > 0, "this shape is meant to have a split tail"
    inp, filt = wl.make_inputs(w)
    a = check_fp32(w, inp, filt)
    b = run_fp32(w, inp, filt)
    np.testing.assert_array_equal(a, b)
    # and the same problem with the split switched off
    mx.set_option("FFMA_STREAMK", 0)
    info, _ = mx.conv_plan_query(d, mx.KERNEL_FP32, sms)
    assert info.split_tiles == 0
    check_fp32(w, inp, filt)


@pytest.mark.parametrize("khc", [1, 2, 3, 5, 7])
@pytest.mark.parametrize("dims", [
    (128, 31, 27, 3, 96, 11, 4, 0, 1.0),     # one pixel per tile: one box per stage
    (128, 31, 27, 3, 128, 11, 4, 0, 1.0),    # 128 filters: the 8 x 8 block on long steps
    (128, 31, 27, 3, 64, 11, 4, 0, 1.0),     # 64 filters: the 4 x 8 block on long steps
    (16, 23, 19, 3, 12, 7, 2, 3, 0.5),       # several pixels per tile: one box per pixel; apron
    (32, 12, 9, 5, 40, 5, 1, 2, 1.0),        # channels in two blocks (3 + 2), stride 1
], ids=lambda s: "x".join(str(v) for v in s))
def test_filter_rows_per_k_step(dims, khc):
    """Few-channel layers take several filter rows per K step; where their number does not
    divide the filter height the last step is short."""
    mx.set_option("FFMA_KH", khc)
    w = wl.Workload("khc", *dims, ("uniform", -1.0, 1.0), ("uniform", -1.0, 1.0), 77)
    info, _ = mx.conv_plan_query(mx.ConvDesc.make(*w.dims), mx.KERNEL_FP32, 148)
    assert info.kwc == w.Sk and 1 <= info.khc <= khc
    check_fp32(w)


@pytest.mark.parametrize("kc", [8, 20, 32, 64, 112])
@pytest.mark.parametrize("dims,tile", [
    ((128, 14, 9, 112, 128, 3, 1, 1, 1.0), (128, 128)),    # 8 x 8 block: steps of up to 112 rows
    ((64, 20, 9, 96, 96, 3, 1, 1, 0.5), (96, 128)),        # 6 x 8 block, four pixels of 32 images
    ((64, 24, 10, 72, 256, 3, 2, 1, 1.0), (128, 256)),     # 8 x 16 block: the ring caps the step at 48 rows
], ids=lambda v: "x".join(str(x) for x in v))
def test_channels_per_k_step(dims, tile, kc):
    """Many-channel layers take as many channels per K step as the tile's ring allows; the
    option pins an upper limit (the planner picks the divisor-friendly count below it)."""
    mx.set_option("FFMA_KC", kc)
    mx.set_option("FFMA_TILE_M", tile[0])
    mx.set_option("FFMA_COLS", tile[1])
    w = wl.Workload("kc", *dims, ("uniform", -1.0, 1.0), ("uniform", -1.0, 1.0), 99)
    info, _ = mx.conv_plan_query(mx.ConvDesc.make(*w.dims), mx.KERNEL_FP32, 148)
    assert info.kwc == 1 and info.kc <= kc and info.stages >= 2
    check_fp32(w)


def test_special_values_fp32():
    """Delta filter reproduces the map bit for bit; permuting filters permutes the output."""
    rng = np.random.default_rng(5)
    Nb, Wi, Hi, Nc = 32, 9, 7, 16
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = np.zeros((Nc, 3, 3, Nc), dtype=np.float32)
    for c in range(Nc):
        filt[c, 1, 1, c] = 1.0
    w = wl.Workload("delta", Nb, Wi, Hi, Nc, Nc, 3, 1, 1, 1.0, None, None, 0)
    got = run_fp32(w, inp, filt)
    np.testing.assert_array_equal(got, inp)


def test_run_to_run_bitwise_identical():
    w = wl.WORKLOADS["mid5x5"].scaled(Nb=128, Wi=9, Hi=9, Nc=32, No=128)
    inp, filt = wl.make_inputs(w)
    a = run_fp32(w, inp, filt)
    b = run_fp32(w, inp, filt)
    np.testing.assert_array_equal(a, b)


# every workload at the size and in the launch configuration that the benchmark times
FULL_SIZE_FP32 = ["first11x11s4", "mid5x5", "wide3x3", "large3x3"] + wl.TABLE1_ORDER


@pytest.mark.parametrize("name", FULL_SIZE_FP32)
def test_full_size_sampled_fp32(name):
    """Benchmark sizes: a band of full output rows plus random single outputs."""
    w = wl.ALL[name]
    inp, filt = wl.make_inputs(w)
    got = run_fp32(w, inp, filt)
    Ho, Wo = got.shape[1:3]
    scale = None
    # full rows: first, one interior, last (cheap for the oracle, covers the apron)
    for y in sorted({0, Ho // 2, Ho - 1}):
        ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha,
                                rows=(y, y + 1))[:, y]
        scale = max(scale or 0.0, float(np.max(np.abs(ref))))
        err = float(np.max(np.abs(got[:, y].astype(np.float64) - ref))) / scale
        assert err <= TOL_FP32, "row %d: E_inf = %.3e" % (y, err)
    rng = np.random.default_rng(1)
    K = w.Nc * w.Sk ** 2
    for _ in range(300):
        o, y, x, n = (int(rng.integers(0, s)) for s in got.shape[:1] + got.shape[1:])
        v, a = oracle.conv_fprop_point(inp, filt, o, y, x, n, stride=w.stride, pad=w.pad,
                                       alpha=w.alpha)
        assert abs(float(got[o, y, x, n]) - v) <= (K + 3) * 2.0 ** -24 * abs(w.alpha) * a + 1e-30
    assert np.isfinite(got).all()


def test_host_entry_point_matches_device_entry_point():
    w = wl.WORKLOADS["tiny3x3"]
    inp, filt = wl.make_inputs(w)
    d = mx.ConvDesc.make(*w.dims)
    ref = run_fp32(w, inp, filt, canary=False)
    h_in = torch.from_numpy(inp).pin_memory()
    h_f = torch.from_numpy(filt).pin_memory()
    h_out = torch.empty(mx.conv_out_elems(d), dtype=torch.float32).pin_memory()
    d_in = torch.empty(inp.size, dtype=torch.float32, device="cuda")
    d_f = torch.empty(filt.size, dtype=torch.float32, device="cuda")
    d_out = torch.empty(h_out.numel(), dtype=torch.float32, device="cuda")
    mx.conv_fprop_host(d, mx.KERNEL_FP32, h_in, h_f, h_out, d_in, d_f, d_out)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(h_out.numpy().reshape(ref.shape), ref)


def test_error_codes_on_device():
    d = mx.ConvDesc.make(32, 8, 8, 4, 32, 3, 1, 1)
    x = torch.zeros(mx.conv_in_elems(d), device="cuda")
    f = torch.zeros(mx.conv_filt_elems(d), device="cuda")
    o = torch.zeros(mx.conv_out_elems(d), device="cuda")
    before = mx.launch_count()
    bad = mx.ConvDesc.make(30, 8, 8, 4, 32, 3, 1, 1)      # Nb not a multiple of 4
    xb = torch.zeros(mx.conv_in_elems(bad), device="cuda")
    ob = torch.zeros(mx.conv_out_elems(bad), device="cuda")
    assert mx.fprop_status(bad, xb, f, ob) == mx.NOT_SUPPORTED
    assert mx.launch_count() == before
    assert mx.fprop_status(d, x, f, o) == mx.OK
    assert mx.launch_count() == before + 1
    # misaligned base pointer
    lib = mx.load_library()
    import ctypes
    st = lib.maxdnn_conv_fprop(ctypes.byref(d), ctypes.c_void_p(x.data_ptr() + 4),
                               ctypes.c_void_p(f.data_ptr()), ctypes.c_void_p(o.data_ptr()), None)
    assert st == mx.INVALID_VALUE
    torch.cuda.synchronize()


# Table 1's ten layer shapes (minibatch 128), reduced in map size / channel count so the
# oracle finishes in seconds but with the paper's filter sizes, strides, paddings and
# filter counts.
TABLE1_REDUCED = {
    "alexnet_conv1": dict(Wi=51, Hi=43),
    "alexnet_conv2": dict(Wi=11, Hi=9),
    "alexnet_conv3": dict(Wi=6, Hi=5, Nc=96),
    "alexnet_conv4": dict(Wi=6, Hi=5, Nc=96),
    "alexnet_conv5": dict(Wi=6, Hi=5, Nc=128),
    "overfeat_L1": dict(Wi=47, Hi=51),
    "overfeat_L2": dict(Wi=10, Hi=9),
    "overfeat_L3": dict(Wi=6, Hi=5, Nc=64),
    "overfeat_L4": dict(Wi=5, Hi=4, Nc=64, No=1024),
    "overfeat_L5": dict(Wi=4, Hi=4, Nc=72, No=1024),
}


@pytest.mark.parametrize("name", wl.TABLE1_ORDER)
def test_table1_layer_shapes_fp32(name):
    check_fp32(wl.TABLE1[name].scaled(**TABLE1_REDUCED[name]))
