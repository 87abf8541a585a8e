"""Times the bf16 tensor-core matrix product of the library on one shape (a small, self-contained case for profilers).

    python -m paper_2204_04179_b200.gemm_probe [--m 32768] [--n 3072] [--k 768] [--layout tn|nn|tt] [--iters 20]

Layouts: tn = A [M,K], B [N,K] (forward); nn = A [M,K], B [K,N] (input gradient); tt = A [K,M], B [K,N]
(weight gradient, fp32 result accumulated, split over K).  Prints one JSON line.
"""
import argparse
import json
import statistics

import torch

from paper_2204_04179_b200 import binding


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--m", type=int, default=32768)
    ap.add_argument("--n", type=int, default=3072)
    ap.add_argument("--k", type=int, default=768)
    ap.add_argument("--layout", default="tn", choices=["tn", "nn", "tt"])
    ap.add_argument("--iters", type=int, default=20)
    args = ap.parse_args()
    dev = "cuda:0"
    cfg = binding.GramConfig(); cfg.n_items = 8; cfg.P_max = 8; cfg.d = 8; cfg.d_ff = 4096
    g = binding.Gram(cfg)
    M, N, K = args.m, args.n, args.k
    a_k, b_k = {"tn": (1, 1), "nn": (1, 0), "tt": (0, 0)}[args.layout]
    A = (torch.randn(M, K, device=dev) * 0.5).to(torch.bfloat16)
    B = (torch.randn(N, K, device=dev) * 0.5).to(torch.bfloat16)
    A = A if a_k else A.T.contiguous()
    B = B if b_k else B.T.contiguous()
    f32 = args.layout == "tt"
    Cm = torch.zeros(M, N, device=dev, dtype=torch.float32 if f32 else torch.bfloat16)
    bias = None if f32 else torch.zeros(N, device=dev)

    def run():
        g.gemm_bf16(A, a_k, B, b_k, Cm, bias, 1 if f32 else 0, M, N, K)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    ts = []
    for _ in range(args.iters):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); run(); e1.record(); torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    ms = statistics.median(ts)
    print(json.dumps({"M": M, "N": N, "K": K, "layout": args.layout, "ms": ms, "TFLOP/s": 2.0 * M * N * K / ms / 1e9}))
    g.close()


if __name__ == "__main__":
    main()
