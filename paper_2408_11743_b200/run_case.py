"""Runs one W4A16 layer shape a few times on the current GPU and prints its average device time.

    python -m paper_2408_11743_b200.run_case --M 16 --K 8192 --N 8192 --G 128 [--iters 20] [--copies 9]
                                             [--sparse] [--check]

A small, self-contained command for timing or profiling one kernel configuration (for example under
`ncu -k regex:gemm`).  Weights rotate over `--copies` packed buffers so that they are read from HBM.
`--check` compares the result with the CPU oracle (test infrastructure) and is off by default.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--M", type=int, default=16)
    ap.add_argument("--K", type=int, default=8192)
    ap.add_argument("--N", type=int, default=8192)
    ap.add_argument("--G", type=int, default=128)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--copies", type=int, default=9)
    ap.add_argument("--sparse", action="store_true")
    ap.add_argument("--check", action="store_true")
    args = ap.parse_args()

    import torch
    import paper_2408_11743_b200 as marlin
    from paper_2408_11743_b200 import inputs, roofline

    M, K, N, G = args.M, args.K, args.N, args.G
    dev = torch.device("cuda")
    if args.sparse:
        case = inputs.make_sparse24(M, K, N, G, seed=1)
        packed0 = marlin.pack_sparse24(torch.from_numpy(case.qc_kpacked.view(np.int32)).to(dev),
                                       torch.from_numpy(case.idx).to(dev), torch.from_numpy(case.S).to(dev), G)
    else:
        case = inputs.make_dense(M, K, N, G, seed=1)
        packed0 = marlin.pack(torch.from_numpy(case.q_kpacked.view(np.int32)).to(dev),
                              torch.from_numpy(case.S).to(dev), G)
    packed = [tuple(t.clone() for t in packed0) for _ in range(args.copies)]
    A = torch.from_numpy(case.A).to(dev)
    C = torch.empty((M, N), dtype=torch.float16, device=dev)
    ws = marlin.new_workspace(M, K, N)

    def run(i):
        p = packed[i % args.copies]
        if args.sparse:
            marlin.gemm_sparse24(A, p[0], p[1], p[2], K, N, G, ws, out=C)
        else:
            marlin.gemm(A, p[0], p[1], K, N, G, ws, out=C)

    for i in range(args.warmup):
        run(i)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.graph(g, stream=s):
        for i in range(args.iters):
            run(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(s):
        g.replay()
        e0.record(s)
        g.replay()
        e1.record(s)
    e1.synchronize()
    t = e0.elapsed_time(e1) * 1e-3 / args.iters
    if marlin.read_status(ws) != 0:
        # a bounded wait inside the kernel expired: the words behind the status word say which one
        rec = ws[:32].cpu().view(torch.int32).tolist()
        print(f"device status {rec[0]}: block {rec[1]} thread {rec[2]} barrier offset {rec[3]} parity {rec[4]} "
              f"polls {rec[5]} waited {rec[6]} us")
        sys.exit(2)
    wb = roofline.weight_bytes(K, N, case.G, sparse24=args.sparse)
    print(f"M={M} K={K} N={N} G={case.G} sparse={args.sparse}: {t * 1e6:.2f} us  "
          f"{wb / t / 1e9:.0f} GB/s weights  {roofline.flops(M, K, N) / t / 1e12:.1f} TFLOP/s")
    if args.check:
        import oracle
        ref = (oracle.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, case.G) if args.sparse
               else oracle.gemm(case.A, case.q_kpacked, case.S, case.G))
        bad, worst, _ = oracle.check_tolerance(C.cpu().numpy(), ref)
        print(f"check: {bad} elements out of tolerance, worst error/allowance {worst:.3f}")
        if bad:
            sys.exit(1)


if __name__ == "__main__":
    main()
