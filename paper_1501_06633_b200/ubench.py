"""Issue-rate microbenchmark of the fp32 inner loop (``csrc/ubench_fp32.cu``).

    python -m paper_1501_06633_b200.ubench            # the whole table
    python -m paper_1501_06633_b200.ubench --one KIND N_LOADS MAP   # one launch (for ncu)
    python -m paper_1501_06633_b200.ubench --stream   # only the bare FFMA2 stream table
    python -m paper_1501_06633_b200.ubench --maps KIND   # one launch per lane map, 6 per row (for ncu)

Per K row of the convolution kernel's 8 x 16 register block a warp issues 64 packed
multiply-adds (FFMA2, two FMA-pipe cycles each) and the loads of 24 operand values.  The
table gives, per variant, the elapsed SM cycles per row and per warp (two warps share a
scheduler, so 128 is the floor), the share of the FMA pipe's peak that leaves, and the
cycles each added instruction costs.  Needs a CUDA device; prints plain text.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "ubench_fp32.cu")
LIB = os.path.join(HERE, "libmaxdnn_ubench.so")
KINDS = {0: "none", 1: "LDS.128", 2: "LDS.64", 3: "LDS.32", 4: "SHFL"}
MAPS = {
    0: "all lanes one word", 1: "lane>>3 (4 words x 8 lanes)", 2: "lane&7 (8 words, per quarter-warp)",
    3: "lane (32 words)", 4: "(lane>>1)&7", 5: "(lane&1)|(lane>>4)<<1", 6: "lane>>2", 7: "lane&3",
    8: "lane>>4", 9: "lane&15", 10: "lane>>1", 11: "lane&1", 12: "(lane>>2)&3",
    13: "(lane&3)|(lane>>4)<<2",
}


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = [os.environ.get("NVCC", "nvcc"), "-std=c++17", "-O3", "-gencode",
               "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC", "-shared",
               "-cudart", "static", "-o", tmp, SRC]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n%s\n%s" % (" ".join(cmd), res.stdout + res.stderr))
        os.replace(tmp, LIB)
    return LIB


def load():
    lib = ctypes.CDLL(build())
    lib.maxdnn_ubench_issue_mix.restype = ctypes.c_int
    lib.maxdnn_ubench_issue_mix.argtypes = [ctypes.c_int] * 5 + [ctypes.c_void_p] * 4
    lib.maxdnn_ubench_ffma2_stream.restype = ctypes.c_int
    lib.maxdnn_ubench_ffma2_stream.argtypes = [ctypes.c_int] * 4 + [ctypes.c_void_p] * 4
    return lib


class Bench:
    def __init__(self):
        import torch
        self.torch = torch
        self.lib = load()
        self.blocks = torch.cuda.get_device_properties(0).multi_processor_count
        g = torch.Generator().manual_seed(1)
        self.seed = (torch.rand(512, generator=g) * 0.5 + 0.25).cuda()
        self.sink = torch.empty(self.blocks * 1024, device="cuda")
        self.cycles = torch.zeros(self.blocks, dtype=torch.int64, device="cuda")

    def run(self, kind, n_loads, lane_map, iters=4096, reps=3):
        """Median over CTAs of the elapsed cycles per K row and per warp (best of `reps`)."""
        best = None
        for _ in range(reps):
            rc = self.lib.maxdnn_ubench_issue_mix(kind, n_loads, lane_map, self.blocks, iters,
                                                  self.seed.data_ptr(), self.sink.data_ptr(),
                                                  self.cycles.data_ptr(), None)
            if rc != 0:
                raise RuntimeError("launch failed: CUDA error %d" % rc)
            self.torch.cuda.synchronize()
            c = float(self.cycles.double().median()) / (iters * 4) / 2.0   # 2 warps per scheduler
            best = c if best is None else min(best, c)
        return best


def stream_table(b):
    """The bare FFMA2 stream: share of the FMA pipe's peak by loop size and warps."""
    print("bare FFMA2 stream (8 accumulators, fixed operands): % of 1 FFMA2 per 2 cycles and scheduler")
    print("%-22s" % "FFMA2 per iteration" + "".join("%9d" % n for n in (32, 64, 128, 256, 512, 1024)))
    for threads in (128, 256, 384, 512, 1024):
        cells = []
        for body in (32, 64, 128, 256, 512, 1024):
            iters = max(64, 262144 // body)
            best = None
            for _ in range(3):
                rc = b.lib.maxdnn_ubench_ffma2_stream(body, threads, b.blocks, iters, b.seed.data_ptr(),
                                                      b.sink.data_ptr(), b.cycles.data_ptr(), None)
                if rc != 0:
                    raise RuntimeError("launch failed: CUDA error %d" % rc)
                b.torch.cuda.synchronize()
                c = float(b.cycles.double().median())
                best = c if best is None else min(best, c)
            wps = threads // 128
            cells.append(100.0 * 2.0 * body * iters * wps / best)
        print("%-22s" % ("%d warps / scheduler" % (threads // 128)) + "".join("%8.1f%%" % c for c in cells))


def main(argv):
    b = Bench()
    if argv[:1] == ["--stream"]:
        stream_table(b)
        return
    if len(argv) >= 4 and argv[0] == "--one":
        kind, nl, mp = int(argv[1]), int(argv[2]), int(argv[3])
        c = b.run(kind, nl, mp, reps=1)
        print("kind %s loads/row %d map %d: %.2f cycles per row per warp" % (KINDS[kind], nl, mp, c))
        return
    if len(argv) >= 2 and argv[0] == "--maps":
        kind = int(argv[1])
        for mp in sorted(MAPS):
            c = b.run(kind, 6, mp, iters=512, reps=1)
            print("kind %s loads/row 6 map %2d %-36s: %.2f cycles per row per warp" % (KINDS[kind], mp, MAPS[mp], c))
        return
    stream_table(b)
    print()
    base = b.run(0, 0, 0)
    print("64 FFMA2 per K row and warp, 2 warps per scheduler: floor 128 cycles per row")
    print("%-10s %-5s %-36s %10s %8s %12s" % ("kind", "n/row", "lane map", "cycles/row", "FMA %", "cycles/instr"))
    print("%-10s %-5d %-36s %10.2f %7.1f%% %12s" % ("none", 0, "order 0: columns outer, serpentine", base, 12800.0 / base, "-"))
    for order, what in ((1, "order 1: filter pairs outer"), (2, "order 2: all P, then all Q"),
                        (3, "order 3: 8 accumulators, one operand pair")):
        c = b.run(0, order, 0)
        print("%-10s %-5d %-36s %10.2f %7.1f%% %12s" % ("none", 0, what, c, 12800.0 / c, "-"))
    for kind in (1, 2, 3, 4):
        for mp in ((0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13) if kind == 1 else (0, 1, 2, 3)):
            for nl in ((2, 4, 6, 8, 12) if mp in (0, 1, 2, 3) else (6,)):
                c = b.run(kind, nl, mp)
                print("%-10s %-5d %-36s %10.2f %7.1f%% %12.2f" % (KINDS[kind], nl, MAPS[mp], c,
                                                                  12800.0 / c, (c - base) / nl))


if __name__ == "__main__":
    main(sys.argv[1:])
