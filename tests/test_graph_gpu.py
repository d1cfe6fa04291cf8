"""The launches are plain stream work (tensor maps travel in kernel parameters, nothing is
allocated or synchronised after the first call), so a sequence of calls can be captured
into a CUDA graph and replayed — the way to run launch-bound small layers."""
import numpy as np
import pytest
import torch

import oracle
import paper_1501_06633_b200 as mx
from paper_1501_06633_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_forward_and_both_gradients_replay_from_a_cuda_graph():
    w = wl.WORKLOADS["tiny3x3"]
    inp, filt = wl.make_inputs(w)
    dout = wl.make_dout(w)
    d = mx.ConvDesc.make(*w.dims)
    x, f, g = (torch.from_numpy(a).cuda() for a in (inp, filt, dout))
    out = torch.zeros(mx.conv_out_elems(d), device="cuda")
    din = torch.zeros(mx.conv_in_elems(d), device="cuda")
    dfilt = torch.zeros(mx.conv_filt_elems(d), device="cuda")
    ws_d = torch.empty(mx.conv_bprop_data_workspace(d), dtype=torch.uint8, device="cuda")
    ws_f = torch.empty(max(16, mx.conv_bprop_filter_workspace(d)), dtype=torch.uint8, device="cuda")

    def run():
        mx.conv_fprop(d, x, f, out)
        mx.conv_bprop_data(d, g, f, din, ws_d)
        mx.conv_bprop_filter(d, x, g, dfilt, ws_f)

    run()                                   # first calls outside the capture (one-time set-up)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            run()
    # new data in the same buffers, results wiped: only a replay can produce them
    inp2, filt2 = wl.make_inputs(w, seed_offset=3)
    dout2 = wl.make_dout(w, seed_offset=3)
    x.copy_(torch.from_numpy(inp2)); f.copy_(torch.from_numpy(filt2)); g.copy_(torch.from_numpy(dout2))
    for t in (out, din, dfilt):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    assert mx.last_device_status() == mx.OK
    refs = (oracle.conv_fprop(inp2, filt2, stride=w.stride, pad=w.pad, alpha=w.alpha),
            oracle.conv_bprop_data(dout2, filt2, (w.Hi, w.Wi), stride=w.stride, pad=w.pad, alpha=w.alpha),
            oracle.conv_bprop_filter(inp2, dout2, w.Sk, stride=w.stride, pad=w.pad, alpha=w.alpha))
    for got_t, ref in zip((out, din, dfilt), refs):
        got = got_t.cpu().numpy().reshape(ref.shape)
        err = float(np.max(np.abs(got.astype(np.float64) - ref))) / float(np.max(np.abs(ref)))
        assert err <= 1e-5
