"""Host-side logic without a GPU: the library loads and exports what the
header declares, descriptors are validated, and the K-step table plus box
geometry of the address-generation stage reproduce the oracle's patch gather
when the copy engine's semantics (boxes, zero fill outside the tensor) are
emulated in numpy."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "maxdnn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(maxdnn_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = mx.load_library()
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(mx.EXPORTED_SYMBOLS)


def test_descriptor_validation_without_gpu():
    lib = mx.load_library()
    good = mx.ConvDesc.make(32, 16, 16, 16, 32, 3, 1, 1)
    assert mx.conv_out_dims(good) == (16, 16)
    assert mx.conv_flops(good) == 76021760
    assert mx.conv_in_elems(good) == 16 * 16 * 16 * 32
    assert mx.conv_filt_elems(good) == 16 * 9 * 32
    assert mx.conv_out_elems(good) == 32 * 16 * 16 * 32
    for bad in [mx.ConvDesc.make(0, 16, 16, 16, 32, 3), mx.ConvDesc.make(32, 16, 16, 16, 32, 3, 0),
                mx.ConvDesc.make(32, 2, 2, 16, 32, 3, 1, 0), mx.ConvDesc.make(32, 16, 16, 16, 32, 3, 1, -1),
                mx.ConvDesc.make(32, 16, 16, 16, 32, 3, 1, 1, float("nan")),
                mx.ConvDesc.make(32, 16, 16, 16, 32, 3, 1, 1, float("inf"))]:
        assert lib.maxdnn_conv_out_dims(ctypes.byref(bad), None, None) == mx.INVALID_VALUE
        assert mx.conv_flops(bad) == 0
        # an invalid descriptor is rejected before any CUDA call is made
        assert lib.maxdnn_conv_fprop(ctypes.byref(bad), None, None, None, None) == mx.INVALID_VALUE
    assert lib.maxdnn_conv_out_dims(None, None, None) == mx.INVALID_VALUE
    assert lib.maxdnn_conv_fprop(ctypes.byref(good), None, None, None, None) == mx.INVALID_VALUE
    assert mx.status_string(mx.NOT_SUPPORTED) == "MAXDNN_NOT_SUPPORTED"
    with pytest.raises(mx.MaxdnnError):
        mx.conv_plan_query(mx.ConvDesc.make(30, 16, 16, 16, 32, 3), mx.KERNEL_FP32, 148)
    with pytest.raises(mx.MaxdnnError):
        mx.conv_plan_query(mx.ConvDesc.make(32, 16, 16, 16, 30, 3), mx.KERNEL_FP32, 148)


def test_flops_match_golden_table():
    for line in open(os.path.join(ROOT, "tests", "golden", "flop_counts.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        Nb, Wi, Hi, Nc, No, Sk, s, p, Ho, Wo, C = map(int, line[1:])
        d = mx.ConvDesc.make(Nb, Wi, Hi, Nc, No, Sk, s, p)
        assert mx.conv_out_dims(d) == (Ho, Wo)
        assert mx.conv_flops(d) == C


def box(arr, starts, sizes):
    """A tiled bulk-tensor load: the box [start, start+size) per axis, zeros
    where it leaves the tensor."""
    out = np.zeros(sizes, dtype=np.float64)
    src, dst = [], []
    for st, sz, ext in zip(starts, sizes, arr.shape):
        lo, hi = max(st, 0), min(st + sz, ext)
        if lo >= hi:
            return out
        src.append(slice(lo, hi))
        dst.append(slice(lo - st, hi - st))
    out[tuple(dst)] = arr[tuple(src)]
    return out


def emulate_fp32_plan(w, inp, filt, sm_count=148):
    d = mx.ConvDesc.make(*w.dims)
    info, steps = mx.conv_plan_query(d, mx.KERNEL_FP32, sm_count)
    Ho, Wo = info.Ho, info.Wo
    Mt, T, Nn, kc, kwc, khc = info.tile_m, info.tile_px, info.tile_n, info.kc, info.kwc, info.khc
    o_blocks = -(-w.No // Mt)
    n_chunks = -(-w.Nb // Nn)
    x_runs = -(-Wo // T)
    assert info.n_tiles == o_blocks * n_chunks * x_runs * Ho
    assert T * Nn <= 256 and Nn % 4 == 0 and Mt in (32, 64, 96, 128, 256)
    assert info.grid == min(info.n_tiles, sm_count)
    # every (c, kh, kw) is covered by exactly one table entry
    seen = np.zeros((w.Nc, w.Sk, w.Sk), dtype=np.int32)
    for s in steps:
        seen[s.c0:s.c0 + kc, s.kh:s.kh + khc, s.kw0:s.kw0 + kwc] += 1   # (clipped at the last row)
        assert s.kw0 + kwc <= w.Sk, "a box must not run past the filter row"
    assert np.all(seen == 1)
    out = np.full((w.No, Ho, Wo, w.Nb), np.nan)
    for tile in range(info.n_tiles):
        r = tile
        ob, r = r % o_blocks, r // o_blocks
        nch, r = r % n_chunks, r // n_chunks
        xr, y = r % x_runs, r // x_runs
        o0, n0, x0 = ob * Mt, nch * Nn, xr * T
        acc = np.zeros((Mt, T, Nn))
        for s in steps:
            A = box(filt, (s.c0, s.kh, s.kw0, o0), (kc, khc, kwc, Mt))         # [c][kh][kw][o]
            for t in range(T):
                Bx = box(inp, (s.c0, y * w.stride - w.pad + s.kh,
                               (x0 + t) * w.stride - w.pad + s.kw0, n0), (kc, khc, kwc, Nn))
                acc[:, t, :] += np.einsum("ckwo,ckwn->on", A, Bx)
        for t in range(T):
            if x0 + t >= Wo:
                continue
            o1, n1 = min(w.No, o0 + Mt), min(w.Nb, n0 + Nn)
            assert np.all(np.isnan(out[o0:o1, y, x0 + t, n0:n1])), "an output is written twice"
            out[o0:o1, y, x0 + t, n0:n1] = w.alpha * acc[:o1 - o0, t, :n1 - n0]
    assert not np.isnan(out).any(), "an output is never written"
    return out


SHAPES = [
    # Nb  Wi  Hi  Nc  No  Sk st pad alpha
    (8, 7, 6, 3, 8, 3, 1, 1, 1.0),
    (132, 5, 4, 9, 100, 3, 1, 1, 0.5),
    (16, 23, 19, 3, 12, 11, 4, 0, 1.0),
    (36, 10, 7, 17, 36, 3, 3, 1, -1.0),
    (20, 13, 4, 33, 68, 2, 1, 0, 1.0),
    (32, 8, 8, 16, 32, 3, 1, 3, 1.0),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_address_generation_reproduces_patch_gather(shape):
    Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha = shape
    w = wl.Workload("plan", Nb, Wi, Hi, Nc, No, Sk, st, pad, alpha, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 77 + Nb)
    inp, filt = wl.make_inputs(w)
    ref = oracle.conv_fprop(inp, filt, stride=st, pad=pad, alpha=alpha)
    got = emulate_fp32_plan(w, inp.astype(np.float64), filt.astype(np.float64))
    assert np.max(np.abs(got - ref)) <= 2.0 ** -22 * max(1.0, np.max(np.abs(ref)))


def test_benchmark_plans_fit_the_device():
    for name in wl.ORDER:
        w = wl.WORKLOADS[name]
        info, steps = mx.conv_plan_query(mx.ConvDesc.make(*w.dims), mx.KERNEL_FP32, 148)
        assert info.smem_bytes <= 227 * 1024 and info.stages >= 2
        assert len(steps) == info.n_ksteps <= 1024
        assert info.grid <= 148
    # the 96-filter first layer gets a 96-high tile (no padded filter rows), the
    # 13x13 layer a tile height that fills whole waves
    assert mx.conv_plan_query(mx.ConvDesc.make(*wl.WORKLOADS["first11x11s4"].dims))[0].tile_m == 96


def test_few_channel_strided_layers_stage_one_strip_per_step():
    """3-channel 11 x 11 stride-4 layers on the tensor kernels: the windows of the tile's
    pixels overlap, so a K step stages one strip of 12 + 4 (pixels - 1) columns instead of
    one 12-column box per pixel, which shows as a smaller stage and a deeper ring; a
    stride-1 few-channel layer (window shift of 4 rows, not a whole swizzle group) keeps
    one box per pixel."""
    d = mx.ConvDesc.make(*wl.WORKLOADS["first11x11s4"].dims)
    bf, _ = mx.conv_plan_query(d, mx.KERNEL_BF16, 148)
    tf, _ = mx.conv_plan_query(d, mx.KERNEL_TF32, 148)
    assert (bf.tile_px, bf.tile_n, bf.kc, bf.n_ksteps * bf.kwc) == (4, 64, 48, 11)
    assert (tf.tile_px, tf.tile_n, tf.kc, tf.n_ksteps * tf.kwc) == (8, 32, 48, 11)
    # stage = 128 filters x 48 rows + strip x 4 channels x 128 B: 24 KB (bf16), 44 KB (tf32)
    assert bf.stages == 8 and tf.stages == 4
    s1, _ = mx.conv_plan_query(mx.ConvDesc.make(64, 14, 11, 1, 32, 3, 1, 1), mx.KERNEL_BF16, 148)
    assert s1.kwc == 1 and s1.kc % 16 == 0


def test_table1_shapes_give_the_printed_output_sizes_and_have_plans():
    """Table 1 prints input size, kernel and output size per layer; the workload list
    must reproduce the output sizes, and every kernel kind must have a plan for them."""
    printed = {"alexnet_conv1": (55, 64), "alexnet_conv2": (27, 192), "alexnet_conv3": (13, 384),
               "alexnet_conv4": (13, 256), "alexnet_conv5": (13, 256), "overfeat_L1": (56, 96),
               "overfeat_L2": (20, 256), "overfeat_L3": (12, 512), "overfeat_L4": (12, 1024),
               "overfeat_L5": (12, 1024)}
    for name, (size, filters) in printed.items():
        w = wl.TABLE1[name]
        d = mx.ConvDesc.make(*w.dims)
        assert mx.conv_out_dims(d) == (size, size) and w.No == filters and w.Nb == 128
        for kind in (mx.KERNEL_FP32, mx.KERNEL_TF32, mx.KERNEL_BF16):
            info, steps = mx.conv_plan_query(d, kind, 148)
            assert info.n_tiles > 0 and info.smem_bytes <= 227 * 1024 and len(steps) == info.n_ksteps


def test_bprop_workspace_sizes_and_refusals(monkeypatch):
    """Host-side planning of the backward entry points (no device needed: the SM count
    is given)."""
    mx.set_option("SM_COUNT", 148)
    d = mx.ConvDesc.make(128, 27, 27, 96, 256, 5, 1, 2, 1.0)
    assert mx.conv_bprop_data_workspace(d, mx.KERNEL_FP32) == 96 * 25 * 256 * 4
    assert mx.conv_bprop_data_workspace(d, mx.KERNEL_BF16) == 96 * 25 * 256 * 2
    strided = mx.ConvDesc.make(128, 227, 227, 3, 96, 11, 4, 0, 1.0)        # stride 4: 16 classes
    r256 = lambda b: (b + 255) // 256 * 256
    # the 16 classes run side by side, each with its own sub-filter bank (3 or 2 taps per
    # axis: nine classes of 3 x 3, six of 3 x 2, one of 2 x 2) and, in fp32, its own dense
    # result (together one din)
    banks = 9 * r256(96 * 9 * 3 * 4) + 6 * r256(96 * 6 * 3 * 4) + r256(96 * 4 * 3 * 4)
    assert mx.conv_bprop_data_workspace(strided) == banks + 3 * 227 * 227 * 128 * 4
    assert mx.conv_bprop_data_workspace(mx.ConvDesc.make(128, 56, 56, 64, 128, 3, 2, 1, 1.0),
                                        mx.KERNEL_BF16) == 64 * 9 * 128 * 2   # stored in place
    for bad in (mx.ConvDesc.make(64, 16, 16, 8, 8, 3, 1, 3, 1.0),):         # pad > Sk - 1
        with pytest.raises(mx.MaxdnnError) as e:
            mx.conv_bprop_data_workspace(bad)
        assert e.value.status == mx.NOT_SUPPORTED
    # filter gradient: partial sums of `splits` reduction splits, or nothing for one split
    kno = 96 * 25 * 256 * 4
    need = mx.conv_bprop_filter_workspace(d)
    assert need % kno == 0 and 2 <= need // kno <= 64          # 40 tiles: the reduction is split
    big = mx.ConvDesc.make(128, 12, 12, 1024, 1024, 3, 1, 1, 1.0)   # 592 tiles: 4 whole waves
    assert mx.conv_bprop_filter_workspace(big) == 0
    assert mx.conv_bprop_filter_workspace(d, mx.KERNEL_BF16) % kno == 0     # 10 channels x 25 taps per tile
    mx.set_option("WGRAD_SPLITS", 5)
    assert mx.conv_bprop_filter_workspace(d) == 5 * kno
    with pytest.raises(mx.MaxdnnError) as e:
        mx.conv_bprop_filter_workspace(mx.ConvDesc.make(30, 16, 16, 8, 8, 3, 1, 1, 1.0))   # Nb % 4
    assert e.value.status == mx.NOT_SUPPORTED


def test_ragged_workspace_sizes():
    """Staging tensors of the relaxed-boundary entry point: Nb and No rounded up to what the
    kernel of each kind needs, each tensor rounded to 256 bytes; nothing for aligned shapes."""
    r256 = lambda b: (b + 255) // 256 * 256
    d = mx.ConvDesc.make(30, 14, 9, 16, 50, 3, 1, 1, 1.0)
    Ho, Wo = 9, 14
    mx.set_option("RAGGED_PADDED", -1)
    assert mx.conv_fprop_ragged_workspace(d, mx.KERNEL_FP32) == 0     # staged inside the kernel
    mx.unset_option("RAGGED_PADDED")
    assert mx.conv_fprop_ragged_workspace(d, mx.KERNEL_FP32) == \
        r256(16 * 9 * 14 * 32 * 4) + r256(16 * 9 * 52 * 4) + r256(52 * Ho * Wo * 32 * 4)
    assert mx.conv_fprop_ragged_workspace(d, mx.KERNEL_BF16) == \
        r256(16 * 9 * 14 * 64 * 2) + r256(16 * 9 * 64 * 2) + r256(64 * Ho * Wo * 64 * 4)
    assert mx.conv_fprop_ragged_workspace(mx.ConvDesc.make(32, 14, 9, 16, 64, 3, 1, 1, 1.0)) == 0
    assert mx.conv_fprop_ragged_workspace(mx.ConvDesc.make(32, 14, 9, 16, 64, 3, 1, 1, 1.0),
                                          mx.KERNEL_BF16) > 0          # bf16 wants 64 images


# ---------------------------------------------------------------------------
# Split tail of the fp32 kernel: the K steps of the last, partly filled wave of tiles are
# dealt out over all CTAs.  Host-only check of the work-item lists.
# ---------------------------------------------------------------------------
SPLIT_SHAPES = [wl.ALL[n].dims for n in ("first11x11s4", "mid5x5", "wide3x3", "large3x3",
                                         "alexnet_conv4", "overfeat_L2", "overfeat_L5")] + [
    (64, 20, 10, 64, 128, 3, 1, 1, 1.0),      # 200 tiles of 128 x 128 (or fewer, larger)
    (128, 13, 13, 40, 96, 3, 1, 1, 1.0),
    (32, 30, 30, 24, 64, 5, 2, 2, 1.0),
]


@pytest.mark.parametrize("dims", SPLIT_SHAPES, ids=lambda s: "x".join(str(v) for v in s))
@pytest.mark.parametrize("sm_count", [148, 132, 7])
def test_split_tail_items_cover_every_k_step_once(dims, sm_count):
    d = mx.ConvDesc.make(*dims)
    info, _ = mx.conv_plan_query(d, mx.KERNEL_FP32, sm_count)
    n = info.n_ksteps
    seen = {}                      # (tile, step) -> cta
    finisher, contributors = {}, {}
    for cta in range(info.grid):
        items = mx.conv_plan_items(d, cta, sm_count)
        kinds = [k for (_, _, _, k) in items]
        assert kinds.count(1) <= 1 and kinds.count(2) <= 1
        if 1 in kinds and 2 in kinds:
            assert kinds.index(1) < kinds.index(2)          # contribute first, then finish
        whole_done = False
        for tile, s0, s1, kind in items:
            assert 0 <= tile < info.n_tiles and 0 <= s0 < s1 <= n
            if kind == 0:
                assert (s0, s1) == (0, n) and not whole_done or tile >= info.n_tiles - info.split_tiles
            else:
                whole_done = True                           # split pieces come after whole tiles
                assert tile >= info.n_tiles - info.split_tiles
            if kind == 1:
                assert s1 < n
                contributors.setdefault(tile, []).append(cta)
            if kind == 2:
                assert s1 == n and s0 > 0
                assert tile not in finisher
                finisher[tile] = cta
            for s in range(s0, s1):
                assert (tile, s) not in seen, "K step computed twice"
                seen[(tile, s)] = cta
    assert len(seen) == info.n_tiles * n, "a K step is missing"
    for tile, ctas in contributors.items():
        assert tile in finisher, "partial sums nobody collects"
        assert max(ctas) < finisher[tile]                   # a finisher waits for lower CTAs only
        # the contributors are exactly the CTAs between the first one and the finisher that
        # have a share at all: their steps are contiguous and ascend with the CTA number
        steps = [(min(s for (t, s), c in seen.items() if t == tile and c == cta), cta) for cta in ctas]
        assert steps == sorted(steps) and [c for _, c in steps] == sorted(ctas)
    for tile in finisher:
        assert tile in contributors
    if info.split_tiles:
        assert 0 < info.split_tiles < info.grid


# ---------------------------------------------------------------------------
# Every kernel instance and plan kind that the planner picks for a benchmarked workload
# must be one that a GPU parity test runs.  The GPU tests' parameter lists are read here
# (planning needs no GPU) and compared with the plans of all fifteen workloads.
# ---------------------------------------------------------------------------
def plan_signature(dims, kind, sms=148):
    d = mx.ConvDesc.make(*dims)
    info, _ = mx.conv_plan_query(d, kind, sms)
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, _ = dims
    if kind == mx.KERNEL_FP32:
        one_box = info.tile_px * info.tile_n == info.tile_cols and \
            (info.tile_px == 1 or (stride == 1 and info.kwc == 1))
        # rows of K per step >= 96: the 8 x 8, 6 x 8 and 4 x 8 blocks then run the instance with the
        # longer main-loop iterations
        long_steps = info.kc * info.kwc * info.khc >= 96 and info.tile_cols == 128 and \
            info.tile_m in (64, 96, 128)
        return ("fp32", info.tile_m, info.tile_cols, one_box, info.kwc > 1, info.khc > 1,
                info.split_tiles > 0, long_steps)
    few = Nc < (8 if kind == mx.KERNEL_TF32 else 16)
    return ("tf32" if kind == mx.KERNEL_TF32 else "bf16", info.pair, info.tile_px * info.tile_n,
            few, info.kwc > 1, stride > 1)


def test_every_benchmarked_plan_is_one_a_gpu_parity_test_runs():
    import test_fprop_gpu as tf
    import test_fprop_tensor_gpu as tt
    # full-size cases: the GPU tests run exactly these workloads (sampled against the oracle)
    fp32_full = set(tf.FULL_SIZE_FP32)
    tensor_full = set(tt.FULL_SIZE_TENSOR) | {("large3x3", "tf32"), ("large3x3", "bf16")}
    for name in wl.ORDER + wl.TABLE1_ORDER:
        w = wl.ALL[name]
        if name != "tiny3x3":
            assert name in fp32_full, name
            for k in ("tf32", "bf16"):
                assert (name, k) in tensor_full, (name, k)
    # and, beyond running the same workload: the same KIND of plan is also compared with the
    # oracle element by element at a reduced size (all outputs, canary strips)
    reduced = set()
    for name, kw in tf.TABLE1_REDUCED.items():
        reduced.add(plan_signature(wl.TABLE1[name].scaled(**kw).dims, mx.KERNEL_FP32))
    for name, kw in [("first11x11s4", dict(Nb=128, Wi=51, Hi=43, No=96)),
                     ("mid5x5", dict(Nb=128, Wi=9, Hi=7, Nc=96, No=256)),
                     ("wide3x3", dict(Nb=128, Wi=6, Hi=5, Nc=256, No=384)),
                     ("large3x3", dict(Nb=64, Wi=14, Hi=9, Nc=128, No=256))]:
        reduced.add(plan_signature(wl.WORKLOADS[name].scaled(**kw).dims, mx.KERNEL_FP32))
    reduced.add(plan_signature(wl.WORKLOADS["tiny3x3"].dims, mx.KERNEL_FP32))
    try:
        for tile_m, cols in [(32, 128), (64, 128), (96, 128), (128, 128), (256, 128), (64, 256),
                             (96, 256), (128, 256)]:
            for stride in (1, 2):
                mx.set_option("FFMA_TILE_M", tile_m)
                mx.set_option("FFMA_COLS", cols)
                reduced.add(plan_signature((64, 11, 8, 24, 296, 3, stride, 1, 1.0), mx.KERNEL_FP32))
        for dims, tile_m, cols in tf.SPLIT:
            mx.reset_options()
            mx.set_option("FFMA_STREAMK", 2)
            if tile_m:
                mx.set_option("FFMA_TILE_M", tile_m)
                mx.set_option("FFMA_COLS", cols)
            reduced.add(plan_signature(dims, mx.KERNEL_FP32))
    finally:
        mx.reset_options()
    missing = []
    for name in wl.ORDER + wl.TABLE1_ORDER:
        sig = plan_signature(wl.ALL[name].dims, mx.KERNEL_FP32)
        # which filter rows / columns a step spans is a property of the shape, not a kernel
        # instance: match on (tile, one box per stage?, split?)
        key = (sig[1], sig[2], sig[3], sig[6], sig[7])
        if key not in {(r[1], r[2], r[3], r[6], r[7]) for r in reduced}:
            missing.append((name, sig))
    assert not missing, "full-size fp32 plans without a reduced-size parity case: %r" % missing
