"""Pins for the CPU oracle: everything here is independent of the oracle's own
code — hand-worked values, brute-force index loops written separately, an
im2col + matmul formulation (Section 3's GEMM statement), a library
convolution, closed forms and invariants of the definition in Section 2."""
import os

import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st

import oracle
from paper_1501_06633_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# independent formulations
# ----------------------------------------------------------------------------
def brute_force(inp, filt, stride, pad, alpha):
    """Seven nested loops over flat buffers with the storage index maps written
    out by hand (python floats are fp64)."""
    Nc, Hi, Wi, Nb = inp.shape
    _, Sk, _, No = filt.shape
    Ho = (Hi + 2 * pad - Sk) // stride + 1
    Wo = (Wi + 2 * pad - Sk) // stride + 1
    fin = [float(v) for v in inp.reshape(-1)]
    ff = [float(v) for v in filt.reshape(-1)]
    out = np.zeros(No * Ho * Wo * Nb, dtype=np.float64)
    for o in range(No):
        for y in range(Ho):
            for x in range(Wo):
                for n in range(Nb):
                    s = 0.0
                    for c in range(Nc):
                        for kh in range(Sk):
                            for kw in range(Sk):
                                h = y * stride - pad + kh
                                w = x * stride - pad + kw
                                if 0 <= h < Hi and 0 <= w < Wi:
                                    s += (ff[((c * Sk + kh) * Sk + kw) * No + o]
                                          * fin[((c * Hi + h) * Wi + w) * Nb + n])
                    out[((o * Ho + y) * Wo + x) * Nb + n] = alpha * s
    return out.reshape(No, Ho, Wo, Nb)


def im2col_matmul(inp, filt, stride, pad, alpha):
    """Section 3: for one output coordinate the Nb x No results are the
    unrolled patch (Nb x Sk^2 Nc) times the filter matrix (Sk^2 Nc x No)."""
    Nc, Hi, Wi, Nb = inp.shape
    _, Sk, _, No = filt.shape
    Ho = (Hi + 2 * pad - Sk) // stride + 1
    Wo = (Wi + 2 * pad - Sk) // stride + 1
    padded = np.zeros((Nc, Hi + 2 * pad + stride, Wi + 2 * pad + stride, Nb), dtype=np.float64)
    padded[:, pad:pad + Hi, pad:pad + Wi, :] = inp
    F = filt.astype(np.float64).reshape(Nc * Sk * Sk, No)        # rows k = (c, kh, kw)
    out = np.zeros((No, Ho, Wo, Nb), dtype=np.float64)
    for y in range(Ho):
        for x in range(Wo):
            patch = padded[:, y * stride:y * stride + Sk, x * stride:x * stride + Sk, :]
            P = patch.reshape(Nc * Sk * Sk, Nb).T                 # Nb x K
            out[:, y, x, :] = alpha * (P @ F).T
    return out


def torch_conv(inp, filt, stride, pad, alpha):
    """Library cross-correlation in fp64 after permuting to NCHW / OIHW."""
    x = torch.from_numpy(np.ascontiguousarray(inp)).double().permute(3, 0, 1, 2)
    w = torch.from_numpy(np.ascontiguousarray(filt)).double().permute(3, 0, 1, 2)
    y = torch.nn.functional.conv2d(x, w, stride=stride, padding=pad)
    return (alpha * y).permute(1, 2, 3, 0).numpy()


def rand_case(rng, Nb, Wi, Hi, Nc, No, Sk):
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = rng.uniform(-1, 1, size=(Nc, Sk, Sk, No)).astype(np.float32)
    return inp, filt


def close(a, b, tol):
    scale = max(float(np.max(np.abs(b))), 1e-30)
    return float(np.max(np.abs(a.astype(np.float64) - b))) / scale <= tol


F32_ROUND = 2.0 ** -23     # one rounding to fp32 on store, relative to the largest value


# ----------------------------------------------------------------------------
# hand-worked examples (tests/golden/hand_worked_conv.txt)
# ----------------------------------------------------------------------------
def _parse_cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "hand_worked_conv.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        key, rest = line.split(None, 1)
        if key == "case":
            cur = {"name": rest.strip()}
            cases.append(cur)
        elif key == "desc":
            cur["desc"] = rest.split()
        else:
            cur[key] = np.array([[float(v) for v in row.split()] for row in rest.split(";")])
    return cases


@pytest.mark.parametrize("case", _parse_cases(), ids=lambda c: c["name"])
def test_hand_worked(case):
    Wi, Hi, Sk, stride, pad = map(int, case["desc"][:5])
    alpha = float(case["desc"][5])
    inp = case["in"].astype(np.float32).reshape(1, Hi, Wi, 1)
    filt = case["filt"].astype(np.float32).reshape(1, Sk, Sk, 1)
    out = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    assert out.shape[1:3] == case["out"].shape
    np.testing.assert_array_equal(out[0, :, :, 0], case["out"].astype(np.float32))


def test_flop_formula_and_out_dims():
    for line in open(os.path.join(GOLDEN, "flop_counts.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        Nb, Wi, Hi, Nc, No, Sk, s, p, Ho, Wo, C = map(int, line[1:])
        assert oracle.out_dims(Nb, Wi, Hi, Nc, No, Sk, s, p) == (Ho, Wo), line[0]
        assert oracle.flops(Nb, Wi, Hi, Nc, No, Sk, s, p) == C, line[0]
    for name in wl.ORDER:  # the generator's shapes are the golden file's shapes
        w = wl.WORKLOADS[name]
        assert oracle.flops(*w.dims) > 0


def test_invalid_descriptors():
    with pytest.raises(ValueError):
        oracle.out_dims(1, 2, 2, 1, 1, 3, 1, 0)      # filter larger than padded map
    with pytest.raises(ValueError):
        oracle.out_dims(1, 4, 4, 1, 1, 3, 0, 0)      # stride 0
    assert oracle.out_dims(1, 2, 2, 1, 1, 3, 1, 1) == (2, 2)


# ----------------------------------------------------------------------------
# brute force / im2col / library on small shapes
# ----------------------------------------------------------------------------
@settings(max_examples=60, deadline=None)
@given(Nb=st.integers(1, 5), Nc=st.integers(1, 4), No=st.integers(1, 5), Sk=st.integers(1, 5),
       extra_w=st.integers(0, 4), extra_h=st.integers(0, 4), stride=st.integers(1, 4),
       pad_frac=st.integers(0, 5), seed=st.integers(0, 2 ** 16),
       alpha=st.sampled_from([1.0, 0.5, -2.0, 0.0]))
def test_matches_brute_force(Nb, Nc, No, Sk, extra_w, extra_h, stride, pad_frac, seed, alpha):
    pad = min(pad_frac, Sk)
    Wi, Hi = max(1, Sk - 2 * pad) + extra_w, max(1, Sk - 2 * pad) + extra_h
    rng = np.random.default_rng(seed)
    inp, filt = rand_case(rng, Nb, Wi, Hi, Nc, No, Sk)
    ref = brute_force(inp, filt, stride, pad, alpha)
    out = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    assert out.shape == ref.shape
    assert close(out, ref, F32_ROUND)


@pytest.mark.parametrize("shape", [
    # Nb Wi Hi Nc No Sk stride pad alpha
    (8, 9, 7, 5, 6, 3, 1, 1, 1.0),
    (4, 23, 19, 3, 8, 11, 4, 0, 1.0),
    (12, 11, 11, 7, 9, 5, 1, 2, 0.5),
    (6, 10, 12, 4, 5, 4, 3, 2, -1.5),
    (3, 6, 6, 2, 2, 1, 2, 0, 1.0),
])
def test_matches_im2col_and_library(shape):
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    rng = np.random.default_rng(7 + Nb)
    inp, filt = rand_case(rng, Nb, Wi, Hi, Nc, No, Sk)
    out = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    assert close(out, im2col_matmul(inp, filt, stride, pad, alpha), F32_ROUND)
    assert close(out, torch_conv(inp, filt, stride, pad, alpha), F32_ROUND)


def test_tiny_workload_matches_library():
    w = wl.WORKLOADS["tiny3x3"]
    inp, filt = wl.make_inputs(w)
    out = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha)
    assert close(out, torch_conv(inp, filt, w.stride, w.pad, w.alpha), F32_ROUND)


def test_scaled_mid_workload_matches_library():
    w = wl.WORKLOADS["mid5x5"].scaled(Nb=16, Nc=12, No=32)
    inp, filt = wl.make_inputs(w)
    out = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha)
    assert close(out, torch_conv(inp, filt, w.stride, w.pad, w.alpha), F32_ROUND)


def test_1x1_is_a_matrix_multiply():
    rng = np.random.default_rng(3)
    Nb, Wi, Hi, Nc, No = 6, 5, 4, 7, 3
    inp, filt = rand_case(rng, Nb, Wi, Hi, Nc, No, 1)
    out = oracle.conv_fprop(inp, filt, stride=1, pad=0, alpha=1.0)
    ref = filt.reshape(Nc, No).astype(np.float64).T @ inp.reshape(Nc, -1).astype(np.float64)
    assert close(out.reshape(No, -1), ref, F32_ROUND)


# ----------------------------------------------------------------------------
# invariants of the definition
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("Sk", [1, 3, 5])
def test_centred_delta_reproduces_input(Sk):
    rng = np.random.default_rng(11)
    Nb, Wi, Hi, Nc = 4, 7, 6, 5
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = np.zeros((Nc, Sk, Sk, Nc), dtype=np.float32)
    for c in range(Nc):
        filt[c, Sk // 2, Sk // 2, c] = 1.0
    out = oracle.conv_fprop(inp, filt, stride=1, pad=Sk // 2, alpha=1.0)
    np.testing.assert_array_equal(out, inp)


def test_linear_in_alpha_and_filters():
    rng = np.random.default_rng(5)
    inp, f1 = rand_case(rng, 4, 8, 8, 3, 5, 3)
    # dyadic values keep every fp32 combination exact, so linearity holds bitwise
    inp = np.round(inp * 64) / 64
    f1 = (np.round(f1 * 64) / 64).astype(np.float32)
    f2 = (np.round(rng.uniform(-1, 1, size=f1.shape) * 64) / 64).astype(np.float32)
    inp = inp.astype(np.float32)
    o1 = oracle.conv_fprop(inp, f1, stride=1, pad=1, alpha=1.0).astype(np.float64)
    o2 = oracle.conv_fprop(inp, f2, stride=1, pad=1, alpha=1.0).astype(np.float64)
    o12 = oracle.conv_fprop(inp, (2 * f1 - 0.5 * f2).astype(np.float32), stride=1, pad=1,
                            alpha=1.0)
    np.testing.assert_array_equal(o12, 2 * o1 - 0.5 * o2)
    oa = oracle.conv_fprop(inp, f1, stride=1, pad=1, alpha=-0.25)
    np.testing.assert_array_equal(oa, -0.25 * o1)
    assert not oracle.conv_fprop(inp, f1, stride=1, pad=1, alpha=0.0).any()


@pytest.mark.parametrize("stride,pad,Sk", [(1, 1, 3), (2, 2, 5), (4, 3, 4), (1, 5, 5)])
def test_padding_equals_explicit_zero_apron(stride, pad, Sk):
    rng = np.random.default_rng(9)
    inp, filt = rand_case(rng, 3, 9, 8, 4, 6, Sk)
    Nc, Hi, Wi, Nb = inp.shape
    padded = np.zeros((Nc, Hi + 2 * pad, Wi + 2 * pad, Nb), dtype=np.float32)
    padded[:, pad:pad + Hi, pad:pad + Wi, :] = inp
    a = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=0.5)
    b = oracle.conv_fprop(padded, filt, stride=stride, pad=0, alpha=0.5)
    np.testing.assert_array_equal(a, b)


def test_translation_batch_and_filter_permutations():
    rng = np.random.default_rng(13)
    stride = 2
    inp, filt = rand_case(rng, 5, 14, 12, 3, 4, 3)
    base = oracle.conv_fprop(inp, filt, stride=stride, pad=0, alpha=1.0)
    shifted = np.zeros_like(inp)
    shifted[:, :, stride:, :] = inp[:, :, :-stride, :]           # move right by one stride
    sh = oracle.conv_fprop(shifted, filt, stride=stride, pad=0, alpha=1.0)
    np.testing.assert_array_equal(sh[:, :, 1:, :], base[:, :, :-1, :])
    pn = rng.permutation(inp.shape[3])
    po = rng.permutation(filt.shape[3])
    perm = oracle.conv_fprop(inp[..., pn], filt[..., po], stride=stride, pad=0, alpha=1.0)
    np.testing.assert_array_equal(perm, base[po][..., pn])


def test_rows_subset_and_point_agree_with_full():
    rng = np.random.default_rng(17)
    inp, filt = rand_case(rng, 4, 9, 9, 3, 5, 3)
    full = oracle.conv_fprop(inp, filt, stride=1, pad=1, alpha=0.5)
    part = oracle.conv_fprop(inp, filt, stride=1, pad=1, alpha=0.5, rows=(2, 5))
    np.testing.assert_array_equal(part[:, 2:5], full[:, 2:5])
    assert not part[:, :2].any() and not part[:, 5:].any()
    ref = brute_force(inp, filt, 1, 1, 0.5)
    for (o, y, x, n) in [(0, 0, 0, 0), (4, 8, 8, 3), (2, 3, 7, 1)]:
        v, a = oracle.conv_fprop_point(inp, filt, o, y, x, n, stride=1, pad=1, alpha=0.5)
        assert abs(v - ref[o, y, x, n]) <= 1e-12 * max(1.0, a)
        assert a >= abs(v) / 0.5 - 1e-12


def test_thread_count_does_not_change_result():
    rng = np.random.default_rng(19)
    inp, filt = rand_case(rng, 8, 10, 10, 4, 6, 3)
    a = oracle.conv_fprop(inp, filt, stride=1, pad=1, nthreads=1)
    b = oracle.conv_fprop(inp, filt, stride=1, pad=1, nthreads=4)
    np.testing.assert_array_equal(a, b)


# ----------------------------------------------------------------------------
# input recipe sanity: interior output variance alpha^2 K sigma_f^2 E[x^2]
# ----------------------------------------------------------------------------
def test_generator_statistics():
    w = wl.WORKLOADS["wide3x3"].scaled(Nb=16, No=64)
    inp, filt = wl.make_inputs(w)
    out = oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha)
    interior = out[:, 1:-1, 1:-1, :].astype(np.float64)
    K = w.Nc * w.Sk ** 2
    expect = w.alpha * (K * 0.01 ** 2 * (1.0 / 3.0)) ** 0.5      # E[x^2] = 1/3 for U[0,1]
    assert abs(interior.std() / expect - 1.0) < 0.05
    again = wl.make_inputs(w)
    np.testing.assert_array_equal(again[0], inp)
    np.testing.assert_array_equal(again[1], filt)
    other = wl.make_inputs(w, seed_offset=1)
    assert not np.array_equal(other[0], inp)


def test_bf16_and_tf32_helpers():
    a = np.array([1.0, 1.00390625, 1.0 + 2 ** -9, 3.14159, -2.5e-3], dtype=np.float32)
    b = wl.from_bf16_bits(wl.to_bf16_bits(a))
    assert np.all(np.abs(b - a) <= np.abs(a) * 2.0 ** -8)
    assert b[0] == 1.0 and b[1] == 1.0        # tie rounds to even
    ref = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(b, ref)
    t = wl.truncate_to_tf32(a)
    assert np.all(np.abs(t) <= np.abs(a)) and np.all(np.abs(t - a) <= np.abs(a) * 2.0 ** -10)


# ----------------------------------------------------------------------------
# per-axis filter size / stride / padding (the relaxed-boundary generalisation)
# ----------------------------------------------------------------------------
def brute_force2(inp, filt, stride, pad, alpha):
    """The sum with separate h / w quantities, index maps by hand, python floats."""
    Nc, Hi, Wi, Nb = inp.shape
    _, Skh, Skw, No = filt.shape
    (sh, sw), (ph, pw) = stride, pad
    Ho = (Hi + 2 * ph - Skh) // sh + 1
    Wo = (Wi + 2 * pw - Skw) // sw + 1
    fin = [float(v) for v in inp.reshape(-1)]
    ff = [float(v) for v in filt.reshape(-1)]
    out = np.zeros(No * Ho * Wo * Nb, dtype=np.float64)
    for o in range(No):
        for y in range(Ho):
            for x in range(Wo):
                for n in range(Nb):
                    s = 0.0
                    for c in range(Nc):
                        for kh in range(Skh):
                            for kw in range(Skw):
                                h = y * sh - ph + kh
                                w = x * sw - pw + kw
                                if 0 <= h < Hi and 0 <= w < Wi:
                                    s += (ff[((c * Skh + kh) * Skw + kw) * No + o]
                                          * fin[((c * Hi + h) * Wi + w) * Nb + n])
                    out[((o * Ho + y) * Wo + x) * Nb + n] = alpha * s
    return out.reshape(No, Ho, Wo, Nb)


RECT_SHAPES = [
    # Nb Wi Hi Nc No Skw Skh (sh, sw) (ph, pw) alpha
    (2, 7, 5, 2, 3, 3, 1, (1, 1), (0, 1), 1.0),        # 1 x 3 row filter
    (2, 6, 8, 1, 2, 2, 5, (2, 1), (2, 0), 0.5),        # 5 x 2, stride 2 down only
    (1, 9, 7, 2, 2, 4, 3, (1, 3), (1, 2), -1.5),
    (3, 5, 5, 2, 2, 3, 3, (2, 2), (1, 1), 1.0),        # square: must equal the square oracle
]


@pytest.mark.parametrize("shape", RECT_SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_per_axis_oracle_matches_brute_force_and_library(shape):
    Nb, Wi, Hi, Nc, No, Skw, Skh, stride, pad, alpha = shape
    rng = np.random.default_rng(31 + Skw * 7 + Skh)
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = rng.uniform(-1, 1, size=(Nc, Skh, Skw, No)).astype(np.float32)
    got = oracle.conv2_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    assert close(got, brute_force2(inp, filt, stride, pad, alpha), 2 * F32_ROUND)
    x = torch.from_numpy(inp).double().permute(3, 0, 1, 2)
    w = torch.from_numpy(filt).double().permute(3, 0, 1, 2)
    lib = (alpha * torch.nn.functional.conv2d(x, w, stride=stride, padding=pad)).permute(1, 2, 3, 0).numpy()
    assert close(got, lib, 2 * F32_ROUND)
    if Skw == Skh and stride[0] == stride[1] and pad[0] == pad[1]:
        np.testing.assert_array_equal(got, oracle.conv_fprop(inp, filt, stride=stride[0], pad=pad[0], alpha=alpha))
