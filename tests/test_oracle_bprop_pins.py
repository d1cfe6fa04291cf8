"""Pins for the BPROP oracle (the two adjoints of Section 2's operation).  Nothing here
uses the oracle's own BPROP code: hand-worked values, brute-force scatter loops (the
literal transpose of the forward sum), adjoint identities against the separately pinned
FPROP oracle, library autograd, closed forms and invariants."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F32_ROUND = 2.0 ** -23


def close(a, b, tol):
    scale = max(float(np.max(np.abs(b))), 1e-30)
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - b))) / scale <= tol


def rand_case(seed, Nb, Wi, Hi, Nc, No, Sk, stride, pad):
    rng = np.random.default_rng(seed)
    Ho = (Hi + 2 * pad - Sk) // stride + 1
    Wo = (Wi + 2 * pad - Sk) // stride + 1
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = rng.uniform(-1, 1, size=(Nc, Sk, Sk, No)).astype(np.float32)
    dout = rng.uniform(-1, 1, size=(No, Ho, Wo, Nb)).astype(np.float32)
    return inp, filt, dout


def scatter_brute_force(inp, filt, dout, stride, pad, alpha):
    """Walk the forward sum term by term (o,y,x,n,c,kh,kw) and add each term's two
    partial derivatives where they belong; flat buffers, index maps written by hand."""
    Nc, Hi, Wi, Nb = inp.shape
    _, Sk, _, No = filt.shape
    _, Ho, Wo, _ = dout.shape
    fin = [float(v) for v in inp.reshape(-1)]
    ff = [float(v) for v in filt.reshape(-1)]
    fg = [float(v) for v in dout.reshape(-1)]
    din = np.zeros(Nc * Hi * Wi * Nb, dtype=np.float64)
    dfilt = np.zeros(Nc * Sk * Sk * No, dtype=np.float64)
    for o in range(No):
        for y in range(Ho):
            for x in range(Wo):
                for n in range(Nb):
                    g = alpha * fg[((o * Ho + y) * Wo + x) * Nb + n]
                    for c in range(Nc):
                        for kh in range(Sk):
                            for kw in range(Sk):
                                h = y * stride - pad + kh
                                w = x * stride - pad + kw
                                if 0 <= h < Hi and 0 <= w < Wi:
                                    i_in = ((c * Hi + h) * Wi + w) * Nb + n
                                    i_f = ((c * Sk + kh) * Sk + kw) * No + o
                                    din[i_in] += ff[i_f] * g
                                    dfilt[i_f] += fin[i_in] * g
    return din.reshape(Nc, Hi, Wi, Nb), dfilt.reshape(Nc, Sk, Sk, No)


def torch_grads(inp, filt, dout, stride, pad, alpha):
    """Library autograd of the library cross-correlation, fp64, NCHW / OIHW."""
    x = torch.from_numpy(np.ascontiguousarray(inp)).double().permute(3, 0, 1, 2).clone().requires_grad_(True)
    w = torch.from_numpy(np.ascontiguousarray(filt)).double().permute(3, 0, 1, 2).clone().requires_grad_(True)
    y = alpha * torch.nn.functional.conv2d(x, w, stride=stride, padding=pad)
    g = torch.from_numpy(np.ascontiguousarray(dout)).double().permute(3, 0, 1, 2)
    y.backward(g)
    return x.grad.permute(1, 2, 3, 0).numpy(), w.grad.permute(1, 2, 3, 0).numpy()


# ----------------------------------------------------------------------------
def _parse_cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "hand_worked_bprop.txt")):
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
    Ho, Wo = case["dout"].shape
    dout = case["dout"].astype(np.float32).reshape(1, Ho, Wo, 1)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    np.testing.assert_array_equal(din[0, :, :, 0], case["din"].astype(np.float32))
    np.testing.assert_array_equal(dfilt[0, :, :, 0], case["dfilt"].astype(np.float32))


SHAPES = [
    # Nb Wi Hi Nc No Sk stride pad alpha
    (2, 5, 4, 2, 3, 3, 1, 1, 1.0),
    (3, 7, 6, 1, 2, 3, 2, 0, 0.5),
    (1, 9, 8, 2, 2, 5, 3, 2, -1.25),
    (2, 6, 6, 3, 1, 2, 2, 1, 1.0),      # even filter, stride = Sk
    (2, 4, 5, 2, 2, 1, 1, 0, 2.0),      # 1x1
    (1, 8, 7, 1, 2, 4, 1, 3, 1.0),      # pad = Sk - 1
    (2, 10, 9, 1, 1, 3, 4, 1, 1.0),     # stride > Sk: some map elements get no gradient
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(str(v) for v in s))
def test_matches_scatter_brute_force(shape):
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    inp, filt, dout = rand_case(7 + Sk * 11 + stride, Nb, Wi, Hi, Nc, No, Sk, stride, pad)
    ref_din, ref_dfilt = scatter_brute_force(inp, filt, dout, stride, pad, alpha)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    assert close(din, ref_din, 2 * F32_ROUND)
    assert close(dfilt, ref_dfilt, 2 * F32_ROUND)


@pytest.mark.parametrize("shape", SHAPES + [(8, 14, 12, 6, 10, 3, 1, 1, 1.0), (4, 23, 19, 3, 8, 11, 4, 0, 1.0),
                                            (8, 13, 13, 8, 12, 5, 1, 2, 0.5)],
                         ids=lambda s: "x".join(str(v) for v in s))
def test_matches_library_autograd(shape):
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    inp, filt, dout = rand_case(101 + Sk, Nb, Wi, Hi, Nc, No, Sk, stride, pad)
    ref_din, ref_dfilt = torch_grads(inp, filt, dout, stride, pad, alpha)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    assert close(din, ref_din, 2 * F32_ROUND)
    assert close(dfilt, ref_dfilt, 2 * F32_ROUND)


@pytest.mark.parametrize("shape", SHAPES + [(16, 15, 11, 5, 7, 3, 2, 1, 0.75)],
                         ids=lambda s: "x".join(str(v) for v in s))
def test_adjoint_identities_against_fprop(shape):
    """<dout, fprop(in, filt)> = <bprop_data(dout, filt), in> = <bprop_filter(in, dout), filt>:
    the three numbers come from three different routines (FPROP is pinned on its own)."""
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = shape
    inp, filt, dout = rand_case(55 + Nb, Nb, Wi, Hi, Nc, No, Sk, stride, pad)
    out = oracle.conv_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    lhs = float(np.sum(dout.astype(np.float64) * out))
    a = float(np.sum(din.astype(np.float64) * inp))
    b = float(np.sum(dfilt.astype(np.float64) * filt))
    scale = float(np.sum(np.abs(dout.astype(np.float64) * out))) + 1e-30
    assert abs(lhs - a) <= 1e-5 * scale
    assert abs(lhs - b) <= 1e-5 * scale


def test_finite_differences_of_the_forward_oracle():
    """d/d(in[i]) and d/d(filt[j]) of <dout, fprop> by central differences: FPROP is
    linear in each argument, so the difference quotient is exact up to rounding."""
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = 2, 6, 5, 2, 3, 3, 2, 1, 0.5
    inp, filt, dout = rand_case(3, Nb, Wi, Hi, Nc, No, Sk, stride, pad)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    g = dout.astype(np.float64)
    rng = np.random.default_rng(9)
    for _ in range(12):
        i = tuple(int(rng.integers(0, s)) for s in inp.shape)
        e = np.zeros_like(inp)
        e[i] = 1.0     # FPROP is linear: <dout, fprop(e_i, filt)> is the derivative itself
        d = float(np.sum(g * oracle.conv_fprop(e, filt, stride=stride, pad=pad, alpha=alpha)))
        assert abs(d - float(din[i])) <= 1e-5 * max(1.0, abs(d))
        j = tuple(int(rng.integers(0, s)) for s in filt.shape)
        e = np.zeros_like(filt)
        e[j] = 1.0
        d = float(np.sum(g * oracle.conv_fprop(inp, e, stride=stride, pad=pad, alpha=alpha)))
        assert abs(d - float(dfilt[j])) <= 1e-5 * max(1.0, abs(d))


def test_1x1_is_two_matrix_multiplies():
    """Sk = 1, stride 1: din = alpha F dout and dfilt = alpha in dout^T as matrices."""
    Nb, Wi, Hi, Nc, No = 4, 5, 3, 6, 7
    inp, filt, dout = rand_case(12, Nb, Wi, Hi, Nc, No, 1, 1, 0)
    alpha = 1.5
    F = filt.astype(np.float64).reshape(Nc, No)
    X = inp.astype(np.float64).reshape(Nc, Hi * Wi * Nb)
    G = dout.astype(np.float64).reshape(No, Hi * Wi * Nb)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, 1, alpha=alpha)
    assert close(din.reshape(Nc, -1), alpha * F @ G, 2 * F32_ROUND)
    assert close(dfilt.reshape(Nc, No), alpha * X @ G.T, 2 * F32_ROUND)


@pytest.mark.parametrize("Sk", [1, 3, 5])
def test_centred_delta_filter_passes_the_gradient_through(Sk):
    Nb, Wi, Hi, Nc = 2, 7, 6, 3
    filt = np.zeros((Nc, Sk, Sk, Nc), dtype=np.float32)
    for c in range(Nc):
        filt[c, Sk // 2, Sk // 2, c] = 1.0
    rng = np.random.default_rng(5)
    dout = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=1, pad=Sk // 2)
    np.testing.assert_array_equal(din, dout)


def test_ones_count_the_terms():
    """in = 1, dout = 1: dfilt[c,kh,kw,o] = alpha Nb x (output pixels whose tap (kh,kw)
    falls inside the map); dout = 1, filt = 1: din[c,h,w,n] = alpha No x (taps reaching (h,w))."""
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = 3, 7, 5, 2, 4, 3, 2, 1, 0.5
    Ho = (Hi + 2 * pad - Sk) // stride + 1
    Wo = (Wi + 2 * pad - Sk) // stride + 1
    ones_in = np.ones((Nc, Hi, Wi, Nb), dtype=np.float32)
    ones_f = np.ones((Nc, Sk, Sk, No), dtype=np.float32)
    ones_g = np.ones((No, Ho, Wo, Nb), dtype=np.float32)
    dfilt = oracle.conv_bprop_filter(ones_in, ones_g, Sk, stride=stride, pad=pad, alpha=alpha)
    din = oracle.conv_bprop_data(ones_g, ones_f, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    for kh in range(Sk):
        for kw in range(Sk):
            cnt = sum(1 for y in range(Ho) for x in range(Wo)
                      if 0 <= y * stride - pad + kh < Hi and 0 <= x * stride - pad + kw < Wi)
            assert np.all(dfilt[:, kh, kw, :] == np.float32(alpha * Nb * cnt))
    for h in range(Hi):
        for w in range(Wi):
            cnt = sum(1 for y in range(Ho) for x in range(Wo) for kh in range(Sk) for kw in range(Sk)
                      if y * stride - pad + kh == h and x * stride - pad + kw == w)
            assert np.all(din[:, h, w, :] == np.float32(alpha * No * cnt))


def test_points_agree_with_full_and_threads_do_not_matter():
    Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha = 4, 9, 8, 3, 5, 3, 2, 1, 0.75
    inp, filt, dout = rand_case(21, Nb, Wi, Hi, Nc, No, Sk, stride, pad)
    din = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha)
    din1 = oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha, nthreads=1)
    dfilt1 = oracle.conv_bprop_filter(inp, dout, Sk, stride=stride, pad=pad, alpha=alpha, nthreads=1)
    np.testing.assert_array_equal(din, din1)
    np.testing.assert_array_equal(dfilt, dfilt1)
    rng = np.random.default_rng(2)
    for _ in range(20):
        c, h, w, n = (int(rng.integers(0, s)) for s in din.shape)
        v, a = oracle.conv_bprop_data_point(dout, filt, (Hi, Wi), c, h, w, n, stride=stride, pad=pad, alpha=alpha)
        assert np.float32(v) == din[c, h, w, n] and a >= abs(v) / abs(alpha) - 1e-12
        c, kh, kw, o = (int(rng.integers(0, s)) for s in dfilt.shape)
        v, a = oracle.conv_bprop_filter_point(inp, dout, Sk, c, kh, kw, o, stride=stride, pad=pad, alpha=alpha)
        assert np.float32(v) == dfilt[c, kh, kw, o] and a >= abs(v) / abs(alpha) - 1e-12


# ----------------------------------------------------------------------------
# per-axis filter size / stride / padding
# ----------------------------------------------------------------------------
RECT = [
    # Nb Wi Hi Nc No Skw Skh (sh, sw) (ph, pw) alpha
    (2, 7, 5, 2, 3, 3, 1, (1, 1), (0, 1), 1.0),
    (2, 6, 8, 1, 2, 2, 5, (2, 1), (2, 0), 0.5),
    (1, 9, 7, 2, 2, 4, 3, (1, 3), (1, 2), -1.5),
    (3, 8, 6, 2, 2, 3, 2, (3, 2), (0, 1), 1.0),
    (3, 5, 5, 2, 2, 3, 3, (2, 2), (1, 1), 1.0),        # square: must equal the square oracle
]


@pytest.mark.parametrize("shape", RECT, ids=lambda s: "x".join(str(v) for v in s))
def test_per_axis_gradients_match_library_autograd_and_adjoint_identities(shape):
    Nb, Wi, Hi, Nc, No, Skw, Skh, stride, pad, alpha = shape
    rng = np.random.default_rng(71 + Skw * 5 + Skh)
    inp = rng.uniform(-1, 1, size=(Nc, Hi, Wi, Nb)).astype(np.float32)
    filt = rng.uniform(-1, 1, size=(Nc, Skh, Skw, No)).astype(np.float32)
    out = oracle.conv2_fprop(inp, filt, stride=stride, pad=pad, alpha=alpha)
    dout = rng.uniform(-1, 1, size=out.shape).astype(np.float32)
    din = oracle.conv2_bprop_data(dout, filt, (Hi, Wi), stride=stride, pad=pad, alpha=alpha)
    dfilt = oracle.conv2_bprop_filter(inp, dout, (Skh, Skw), stride=stride, pad=pad, alpha=alpha)
    # library autograd, fp64
    x = torch.from_numpy(inp).double().permute(3, 0, 1, 2).clone().requires_grad_(True)
    w = torch.from_numpy(filt).double().permute(3, 0, 1, 2).clone().requires_grad_(True)
    y = alpha * torch.nn.functional.conv2d(x, w, stride=stride, padding=pad)
    y.backward(torch.from_numpy(dout).double().permute(3, 0, 1, 2))
    assert close(din, x.grad.permute(1, 2, 3, 0).numpy(), 2 * F32_ROUND)
    assert close(dfilt, w.grad.permute(1, 2, 3, 0).numpy(), 2 * F32_ROUND)
    # adjoint identities against the per-axis forward oracle (pinned on its own)
    lhs = float(np.sum(dout.astype(np.float64) * out))
    scale = float(np.sum(np.abs(dout.astype(np.float64) * out))) + 1e-30
    assert abs(lhs - float(np.sum(din.astype(np.float64) * inp))) <= 1e-5 * scale
    assert abs(lhs - float(np.sum(dfilt.astype(np.float64) * filt))) <= 1e-5 * scale
    if Skw == Skh and stride[0] == stride[1] and pad[0] == pad[1]:
        np.testing.assert_array_equal(din, oracle.conv_bprop_data(dout, filt, (Hi, Wi), stride=stride[0],
                                                                  pad=pad[0], alpha=alpha))
        np.testing.assert_array_equal(dfilt, oracle.conv_bprop_filter(inp, dout, Skh, stride=stride[0],
                                                                      pad=pad[0], alpha=alpha))
