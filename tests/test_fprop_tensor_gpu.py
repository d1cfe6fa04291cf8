"""GPU parity of the tensor-core (tcgen05) path against the CPU oracle.

Two comparisons per case.  Primary: against the oracle on the ORIGINAL fp32
inputs, within the tolerance stated for the arithmetic (TF32 5e-3, BF16 2e-2 of
the largest output).  Secondary: against the oracle on inputs rounded the way
the kernel's operands are (fp32 with the low 13 mantissa bits cleared for TF32,
bf16 values for BF16); what is left is fp32 accumulation order, 1e-5."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"tf32": 5e-3, "bf16": 2e-2}
TOL_ROUNDED = 1e-5
KIND = {"tf32": mx.KERNEL_TF32, "bf16": mx.KERNEL_BF16}


def device_inputs(kernel, inp, filt):
    if kernel == "bf16":
        to_dev = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        rounded = lambda a: wl.from_bf16_bits(wl.to_bf16_bits(a))
    else:
        to_dev = lambda a: torch.from_numpy(a).cuda()
        rounded = wl.truncate_to_tf32
    return to_dev(inp), to_dev(filt), rounded(inp), rounded(filt)


def run(kernel, w, inp, filt):
    d = mx.ConvDesc.make(*w.dims)
    d_in, d_f, r_in, r_f = device_inputs(kernel, inp, filt)
    n_out = mx.conv_out_elems(d)
    guard = 1024
    buf = torch.full((n_out + 2 * guard,), 12345.0, dtype=torch.float32, device="cuda")
    fn = mx.conv_fprop_tf32 if kernel == "tf32" else mx.conv_fprop_bf16
    fn(d, d_in, d_f, buf[guard:guard + n_out])
    assert mx.last_device_status() == mx.OK
    host = buf.cpu().numpy()
    assert np.all(host[:guard] == 12345.0) and np.all(host[guard + n_out:] == 12345.0)
    Ho, Wo = mx.conv_out_dims(d)
    return host[guard:guard + n_out].reshape(w.No, Ho, Wo, w.Nb), r_in, r_f


def rel_inf(g, r):
    return float(np.max(np.abs(g.astype(np.float64) - r.astype(np.float64)))) / \
        max(float(np.max(np.abs(r))), 1e-30)


def check(kernel, w, inp=None, filt=None):
    if inp is None:
        inp, filt = wl.make_inputs(w)
    got, r_in, r_f = run(kernel, w, inp, filt)
    ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha)
    ref_rounded = oracle.conv_fprop(r_in, r_f, stride=w.stride, pad=w.pad, alpha=w.alpha)
    assert got.shape == ref.shape
    e1, e2 = rel_inf(got, ref), rel_inf(got, ref_rounded)
    assert e1 <= TOL[kernel], "%s vs oracle: E_inf = %.3e" % (kernel, e1)
    assert e2 <= TOL_ROUNDED, "%s vs oracle on rounded inputs: E_inf = %.3e" % (kernel, e2)


SCALED = [
    ("large3x3", dict(Nb=64, Wi=14, Hi=9, Nc=128, No=256)),
    ("large3x3", dict(Nb=64, Wi=13, Hi=5, Nc=72, No=160)),      # ragged x tail, channel tail
    ("mid5x5", dict(Nb=128, Wi=9, Hi=7, Nc=96, No=256)),
    ("wide3x3", dict(Nb=128, Wi=6, Hi=5, Nc=256, No=384)),
    ("first11x11s4", dict(Nb=128, Wi=51, Hi=43, Nc=3, No=96)),  # stride 4: one box per pixel
]


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
@pytest.mark.parametrize("name,kw", SCALED)
def test_scaled_workloads(kernel, name, kw):
    check(kernel, wl.WORKLOADS[name].scaled(**kw))


def test_tiny_workload_tf32():
    check("tf32", wl.WORKLOADS["tiny3x3"])


EDGE = [
    # Nb  Wi  Hi  Nc  No  Sk st pad alpha
    (64, 5, 5, 1, 32, 1, 1, 0, 1.0),         # one channel, 1x1 filter
    (64, 7, 6, 3, 32, 3, 1, 1, -2.0),        # few channels: mostly zero-filled K rows
    (64, 9, 9, 20, 96, 5, 2, 2, 1.0),        # stride 2 with padding, 96 filters in a 128 tile
    (320, 6, 5, 9, 64, 3, 1, 1, 0.5),        # more images than one tile holds
    (192, 10, 7, 17, 160, 3, 3, 1, 1.0),     # 192 images: ragged image chunk
    (64, 5, 5, 8, 32, 5, 1, 0, 1.0),         # single output pixel
    (64, 8, 8, 16, 32, 3, 1, 3, 1.0),        # all-apron patches
    (128, 4, 4, 12, 32, 3, 1, 1, 0.0),       # alpha = 0
    (64, 30, 3, 5, 64, 3, 1, 1, 1.0),        # wide short map
]


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
@pytest.mark.parametrize("shape", EDGE, ids=lambda s: "x".join(str(v) for v in s))
def test_edge_shapes(kernel, shape):
    Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha = shape
    w = wl.Workload("edge", Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 777 + Nb + No)
    check(kernel, w)


def test_tf32_on_32_images():
    w = wl.Workload("edge", 32, 9, 7, 24, 64, 3, 1, 1, 1.0, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 31)
    check("tf32", w)


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
def test_full_size_large3x3_sampled(kernel):
    """The benchmark's 3x3 layer at full size: three full output rows and random
    single outputs against the oracle."""
    w = wl.WORKLOADS["large3x3"]
    inp, filt = wl.make_inputs(w)
    got, r_in, r_f = run(kernel, w, inp, filt)
    Ho = got.shape[1]
    for y in sorted({0, Ho // 2, Ho - 1}):
        ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha,
                                rows=(y, y + 1))[:, y]
        refr = oracle.conv_fprop(r_in, r_f, stride=w.stride, pad=w.pad, alpha=w.alpha,
                                 rows=(y, y + 1))[:, y]
        assert rel_inf(got[:, y], ref) <= TOL[kernel]
        assert rel_inf(got[:, y], refr) <= TOL_ROUNDED
    rng = np.random.default_rng(2)
    scale = float(np.max(np.abs(got)))
    for _ in range(300):
        o, y, x, n = (int(rng.integers(0, s)) for s in got.shape)
        v, _ = oracle.conv_fprop_point(r_in, r_f, o, y, x, n, stride=w.stride, pad=w.pad,
                                       alpha=w.alpha)
        assert abs(float(got[o, y, x, n]) - v) <= TOL_ROUNDED * scale
    assert np.isfinite(got).all()


# every workload at full size through both operand types (large3x3 has its own test above):
# filter columns merged into K (the 3-channel layers), two-SM tiles with images split and
# strips of 5 columns (5 x 5), one-SM tiles for 384 filters, 192-column tiles (13 x 13), ...
FULL_SIZE_TENSOR = [(n, k) for n in ["first11x11s4", "mid5x5", "wide3x3"] + wl.TABLE1_ORDER
                    for k in ("tf32", "bf16")]


def tol_rounded_long_k(K):
    """Against the oracle on rounded operands what is left is the fp32 accumulation: order of
    summation (1e-5) and, on the tensor cores, the accumulator being truncated at every MMA —
    a one-sided error that grows with the length of a sum of same-signed terms (maps in
    [0, 1)): measured 1.0e-8 K of the largest output, allowed 1.5e-8 K."""
    return max(TOL_ROUNDED, 1.5e-8 * K)


@pytest.mark.parametrize("name,kernel", FULL_SIZE_TENSOR)
def test_full_size_sampled_in_the_benchmarked_plans(name, kernel):
    """Every kind of plan the planner picks at full size (the launch configuration the bench
    and the Table 1 run time): first / middle / last output row and random single outputs."""
    w = wl.ALL[name]
    inp, filt = wl.make_inputs(w)
    got, r_in, r_f = run(kernel, w, inp, filt)
    assert np.isfinite(got).all()
    Ho = got.shape[1]
    scale = float(np.max(np.abs(got)))
    tol_r = tol_rounded_long_k(w.Nc * w.Sk * w.Sk)
    for y in sorted({0, Ho // 2, Ho - 1}):
        ref = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha,
                                rows=(y, y + 1))[:, y]
        refr = oracle.conv_fprop(r_in, r_f, stride=w.stride, pad=w.pad, alpha=w.alpha,
                                 rows=(y, y + 1))[:, y]
        # the stated tolerance of the arithmetic, against the oracle on the original inputs
        assert float(np.max(np.abs(got[:, y].astype(np.float64) - ref))) <= TOL[kernel] * scale
        assert float(np.max(np.abs(got[:, y].astype(np.float64) - refr))) <= tol_r * scale
    rng = np.random.default_rng(3)
    for _ in range(200):
        o, y, x, n = (int(rng.integers(0, s)) for s in got.shape)
        v, _ = oracle.conv_fprop_point(r_in, r_f, o, y, x, n, stride=w.stride, pad=w.pad,
                                       alpha=w.alpha)
        assert abs(float(got[o, y, x, n]) - v) <= tol_r * scale


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
def test_run_to_run_bitwise_identical(kernel):
    w = wl.WORKLOADS["large3x3"].scaled(Nb=64, Wi=12, Hi=8, Nc=64, No=128)
    inp, filt = wl.make_inputs(w)
    a, _, _ = run(kernel, w, inp, filt)
    b, _, _ = run(kernel, w, inp, filt)
    np.testing.assert_array_equal(a, b)


def test_unsupported_shapes_launch_nothing():
    before = mx.launch_count()
    for kind, Nb, No in [(mx.KERNEL_TF32, 48, 64), (mx.KERNEL_BF16, 32, 64), (mx.KERNEL_TF32, 64, 48)]:
        d = mx.ConvDesc.make(Nb, 8, 8, 8, No, 3, 1, 1)
        eb = torch.bfloat16 if kind == mx.KERNEL_BF16 else torch.float32
        x = torch.zeros(mx.conv_in_elems(d), device="cuda", dtype=eb)
        f = torch.zeros(mx.conv_filt_elems(d), device="cuda", dtype=eb)
        o = torch.zeros(mx.conv_out_elems(d), device="cuda")
        assert mx.fprop_status(d, x, f, o, kind) == mx.NOT_SUPPORTED
    assert mx.launch_count() == before


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
    "overfeat_L5": dict(Wi=4, Hi=4, Nc=80, No=1024),
}


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
@pytest.mark.parametrize("name", list(TABLE1_REDUCED))
def test_table1_layer_shapes(kernel, name):
    """Table 1's layer shapes (reduced maps / channels) through the tensor-core path."""
    check(kernel, wl.TABLE1[name].scaled(**TABLE1_REDUCED[name]))


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
@pytest.mark.parametrize("khc", [0, 2])
@pytest.mark.parametrize("shape", [
    (128, 47, 39, 3, 96, 11, 4, 0, 1.0),      # the first-layer shape: 12 columns x 4 channels = 48 K rows
    (64, 23, 19, 3, 64, 11, 4, 2, 0.5),       # with padding: windows reach into the apron
    (64, 14, 11, 1, 32, 3, 1, 1, 1.0),        # one channel, stride 1: overlapping windows per pixel
    (64, 12, 9, 5, 160, 5, 2, 2, 1.0),        # 5 channels -> boxes of 8, stride 2
    (128, 9, 9, 7, 32, 7, 1, 3, 1.0),         # 7 x 7 x 7
    (64, 10, 8, 2, 32, 2, 1, 0, 1.0),         # 2 x 2 filter, 2 channels
], ids=lambda s: "x".join(str(v) for v in s))
def test_few_channel_layers_merge_filter_columns_into_k(kernel, shape, khc, monkeypatch):
    """Layers with fewer channels than the MMA's K take K steps that span all filter columns
    (and khc filter rows) of a few channels; surplus K rows are out-of-bounds zeros."""
    if khc:
        mx.set_option("UMMA_MERGE", khc)
    Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha = shape
    w = wl.Workload("merged", Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 8800 + Sk)
    d = mx.ConvDesc.make(*w.dims)
    try:
        info, _ = mx.conv_plan_query(d, KIND[kernel], 148)
    except mx.MaxdnnError:
        assert khc                       # only a forced step size may not fit shared memory
        pytest.skip("two filter rows per step do not fit two stages for this shape")
    # merged plan taken: a step spans whole filter rows (with the shared strip of a strided
    # layer, kwc counts the filter rows of a step and kc the K rows of one)
    assert info.kc >= Nc * Sk and info.n_ksteps * info.kwc < Sk + info.kwc and info.n_ksteps <= Sk
    check(kernel, w)


@pytest.mark.parametrize("kernel", ["tf32", "bf16"])
@pytest.mark.parametrize("shape", [
    (64, 14, 9, 128, 256, 3, 1, 1, 1.0),      # strip reuse, two tiles of 256 filters
    (128, 9, 7, 96, 256, 5, 1, 2, 1.0),       # the CTAs of the pair split the images
    (256, 7, 5, 48, 256, 3, 1, 1, 1.0),       # one pixel x 256 images per tile, split by image
    (32, 21, 5, 40, 256, 3, 1, 1, 1.0),       # tf32 only: 8 pixels x 32 images, split by pixel
    (64, 13, 5, 72, 512, 3, 1, 1, 0.5),       # ragged pixel tail, channel tail
    (128, 23, 19, 16, 256, 11, 4, 0, 1.0),    # stride 4: one box per pixel
    (64, 12, 6, 24, 160, 3, 1, 1, 1.0),       # 160 filters: second CTA of the pair mostly idle
], ids=lambda s: "x".join(str(v) for v in s))
def test_two_sm_tiles(kernel, shape, monkeypatch):
    """The two-SM variant (256 filters per CTA pair, cta_group::2 MMAs), taken only on
    request, against the oracle."""
    mx.set_option("UMMA_PAIR", 1)
    Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha = shape
    if kernel == "bf16" and Nb % 64 != 0:
        pytest.skip("bf16 tiles hold whole groups of 64 images")
    w = wl.Workload("pair", Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 4321 + No)
    d = mx.ConvDesc.make(*w.dims)
    info, _ = mx.conv_plan_query(d, KIND[kernel], 148)
    assert info.tile_m == 256 and info.grid % 2 == 0
    check(kernel, w)
