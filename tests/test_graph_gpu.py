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


@pytest.mark.parametrize("kernel", ["fp32", "bf16"])
def test_strided_map_gradient_forks_and_joins(kernel):
    """Stride 2: the four residue classes run on the caller's stream and on the library's
    side streams.  (a) Work queued on the caller's stream before and after the call is
    ordered with all classes: the inputs are written by a kernel just before the call and
    the result is consumed by a kernel just after it, with no host synchronisation.  (b)
    The same call captured into a CUDA graph (fork and join by events) replays correctly."""
    kind = {"fp32": mx.KERNEL_FP32, "bf16": mx.KERNEL_BF16}[kernel]
    tol = {"fp32": 1e-5, "bf16": 2e-2}[kernel]
    w = wl.Workload("s2", 64, 20, 14, 32, 64, 3, 2, 1, 1.0, ("uniform", -1.0, 1.0),
                    ("uniform", -1.0, 1.0), 7700)
    d = mx.ConvDesc.make(*w.dims)
    _, filt = wl.make_inputs(w)
    dout = wl.make_dout(w)
    dt = torch.bfloat16 if kernel == "bf16" else torch.float32
    if kernel == "bf16":
        filt = wl.from_bf16_bits(wl.to_bf16_bits(filt))
        dout = wl.from_bf16_bits(wl.to_bf16_bits(dout))
    ref = oracle.conv_bprop_data(dout, filt, (w.Hi, w.Wi), stride=2, pad=1, alpha=1.0)
    scale = float(np.max(np.abs(ref)))
    f = torch.from_numpy(filt).cuda().to(dt)
    g_src = torch.from_numpy(dout).cuda().to(dt)
    g = torch.zeros_like(g_src)
    din = torch.zeros(mx.conv_in_elems(d), device="cuda")
    total = torch.zeros(mx.conv_in_elems(d), device="cuda")
    ws = torch.empty(mx.conv_bprop_data_workspace(d, kind), dtype=torch.uint8, device="cuda")
    mx.conv_bprop_data(d, g, f, din, ws, kind)          # one-time set-up outside any capture
    torch.cuda.synchronize()

    side = torch.cuda.Stream()

    def run():
        g.copy_(g_src)                                  # producer on the same stream
        mx.conv_bprop_data(d, g, f, din, ws, kind, stream=side)
        total.copy_(din)                                # consumer on the same stream

    with torch.cuda.stream(side):
        g.zero_(); din.fill_(float("nan")); total.zero_()
        run()
    side.synchronize()
    assert mx.last_device_status() == mx.OK
    got = total.cpu().numpy().reshape(ref.shape)
    assert float(np.max(np.abs(got - ref))) <= tol * scale

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            run()
    g.zero_(); din.fill_(float("nan")); total.zero_()
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    assert mx.last_device_status() == mx.OK
    got = total.cpu().numpy().reshape(ref.shape)
    assert float(np.max(np.abs(got - ref))) <= tol * scale


def test_strided_map_gradient_from_two_host_threads():
    """Two host threads, each with its own stream and buffers, call the strided map gradient
    (which borrows the library's side streams and events) at the same time: the fork / join
    sequences must not mix."""
    import threading
    shapes = [(64, 15, 11, 32, 64, 3, 2, 1, 1.0), (64, 23, 19, 32, 64, 7, 4, 3, 1.0)]
    cases = []
    for i, s in enumerate(shapes):
        w = wl.Workload("mt", *s, ("uniform", -1.0, 1.0), ("uniform", -1.0, 1.0), 5100 + i)
        _, filt = wl.make_inputs(w)
        dout = wl.make_dout(w)
        d = mx.ConvDesc.make(*w.dims)
        ref = oracle.conv_bprop_data(dout, filt, (w.Hi, w.Wi), stride=w.stride, pad=w.pad, alpha=w.alpha)
        cases.append((d, torch.from_numpy(dout).cuda(), torch.from_numpy(filt).cuda(), ref,
                      torch.empty(mx.conv_bprop_data_workspace(d), dtype=torch.uint8, device="cuda"),
                      torch.empty(mx.conv_in_elems(d), device="cuda")))
    for c in cases:                                      # one-time set-up on this thread
        mx.conv_bprop_data(c[0], c[1], c[2], c[5], c[4])
    torch.cuda.synchronize()
    errs = []

    def worker(tid):
        torch.cuda.set_device(0)
        st = torch.cuda.Stream()
        d, g, f, ref, ws, din = cases[tid]
        for it in range(40):
            with torch.cuda.stream(st):
                din.fill_(float("nan"))
                mx.conv_bprop_data(d, g, f, din, ws, stream=st)
                got = din.cpu().numpy().reshape(ref.shape)
            e = float(np.max(np.abs(got - ref))) / float(np.max(np.abs(ref)))
            if not e <= 1e-5:
                errs.append((tid, it, e))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errs, errs[:3]
    assert mx.last_device_status() == mx.OK
