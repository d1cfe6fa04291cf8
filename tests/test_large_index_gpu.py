"""Maximum sizes: an output tensor of more than 2^31 elements (12.9 GB) — element offsets do
not fit 32 bits anywhere on the path.  Sampled outputs against the oracle's single-point
routine (values are fetched from the device one by one; the tensor is never copied)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kernel", ["fp32", "bf16"])
def test_output_beyond_2_31_elements(kernel):
    free, _ = torch.cuda.mem_get_info()
    if free < 20 * 2 ** 30:
        pytest.skip("needs 20 GB of free device memory")
    w = wl.Workload("huge", 128, 512, 512, 4, 96, 3, 1, 1, 1.0, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 777)
    d = mx.ConvDesc.make(*w.dims)
    n_out = mx.conv_out_elems(d)
    assert n_out > 2 ** 31
    inp, filt = wl.make_inputs(w)
    if kernel == "bf16":
        to_dev = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        r_in, r_f = wl.from_bf16_bits(wl.to_bf16_bits(inp)), wl.from_bf16_bits(wl.to_bf16_bits(filt))
        kind, tol = mx.KERNEL_BF16, 1e-5
    else:
        to_dev = lambda a: torch.from_numpy(a).cuda()
        r_in, r_f = inp, filt
        kind, tol = mx.KERNEL_FP32, 1e-5
    out = torch.empty(n_out, dtype=torch.float32, device="cuda")
    out[-1024:] = float("nan")
    out[:1024] = float("nan")
    assert mx.fprop_status(d, to_dev(inp), to_dev(filt), out, kind) == mx.OK
    assert mx.last_device_status() == mx.OK
    Ho, Wo = mx.conv_out_dims(d)
    rng = np.random.default_rng(8)
    pts = [(int(rng.integers(0, w.No)), int(rng.integers(0, Ho)), int(rng.integers(0, Wo)),
            int(rng.integers(0, w.Nb))) for _ in range(150)]
    pts += [(0, 0, 0, 0), (w.No - 1, Ho - 1, Wo - 1, w.Nb - 1), (w.No - 1, 0, Wo - 1, 5),
            (w.No // 2, Ho - 1, 0, w.Nb - 1)]                     # corners: first / last element
    idx = torch.tensor([((o * Ho + y) * Wo + x) * w.Nb + n for o, y, x, n in pts], device="cuda")
    assert int(idx.max()) > 2 ** 31
    got = out[idx].cpu().numpy()
    scale = 0.0
    refs = []
    for o, y, x, n in pts:
        v, _ = oracle.conv_fprop_point(r_in, r_f, o, y, x, n, stride=1, pad=1, alpha=1.0)
        refs.append(v)
        scale = max(scale, abs(v))
    assert np.all(np.isfinite(got))
    assert float(np.max(np.abs(got - np.array(refs)))) <= tol * scale
    del out
    torch.cuda.empty_cache()
