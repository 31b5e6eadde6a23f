"""Run a few launches of one cq_gemm case (for ncu captures and quick timing).

    python profile_case.py --B 4 --G 128 --N 8192 --K 8192 --M 1 --mode 0 --launches 12

Weights rotate over enough copies that no launch finds them in L2.  Prints the CUDA-event time per
launch.  Inputs are the seeded synthetic tensors the benchmark uses.
"""
import argparse
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import datagen  # noqa: E402
import paper_2608_06763_b200 as cq  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    for name, default in (("B", 4), ("G", 128), ("N", 8192), ("K", 8192), ("M", 1), ("mode", 0), ("launches", 12),
                          ("copies", 0), ("graph", 1)):
        ap.add_argument("--" + name, type=int, default=default)
    a = ap.parse_args()
    k, s, aa, bb = datagen.logical_quantized(a.N, a.K, a.B, a.G, 1, name="profile")
    codes = cq.cq_pack_codes(torch.from_numpy(k).cuda(), a.B)
    pw = cq.cq_repack(codes, torch.from_numpy(s).cuda(), torch.from_numpy(np.ascontiguousarray(aa)).cuda(),
                      torch.from_numpy(np.ascontiguousarray(bb)).cuda(), a.B, a.G, a.N, a.K)
    nbytes = pw.layout.numel()
    copies = a.copies or min(int(np.ceil(2 * 126 * 2 ** 20 / nbytes)) + 1, 24)
    pws = [pw] + [cq.PackedWeights(pw.layout.clone(), a.B, a.G, a.N, a.K) for _ in range(copies - 1)]
    x = torch.from_numpy(datagen.activations(a.M, a.K, seed=1).view(np.int16)).cuda().view(torch.bfloat16)
    ws = torch.zeros(cq.cq_workspace_bytes(a.B, a.G, a.M, a.N, a.K, a.mode), dtype=torch.uint8, device="cuda")
    y = torch.empty((a.M, a.N), dtype=torch.bfloat16, device="cuda")
    for i in range(3):
        cq.cq_gemm(pws[i % copies], x, a.mode, ws, y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(a.launches):
        cq.cq_gemm(pws[(i + 3) % copies], x, a.mode, ws, y)
    e1.record()
    torch.cuda.synchronize()
    us_host = e0.elapsed_time(e1) * 1e3 / a.launches
    us = us_host
    if a.graph:
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                for i in range(a.launches):
                    cq.cq_gemm(pws[i % copies], x, a.mode, ws, y)
            g.replay()
            st.synchronize()
            best = 1e30
            for _ in range(3):
                e0.record(st)
                g.replay()
                e1.record(st)
                st.synchronize()
                best = min(best, e0.elapsed_time(e1) * 1e3 / a.launches)
        us = best
    eff = a.N * a.K * (a.B + 64.0 / a.G) / 8.0
    print(f"B={a.B} G={a.G} N={a.N} K={a.K} M={a.M} mode={a.mode}: {us:.2f} us/launch in a CUDA graph ({us_host:.2f} host-launched), "
          f"{eff / us / 1e3:.1f} GB/s effective, {2.0 * a.M * a.N * a.K / us / 1e6:.2f} TFLOP/s")


if __name__ == "__main__":
    main()
