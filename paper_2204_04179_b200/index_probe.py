"""Times dedup, gather and accumulate alone on one sweep cell (seeded Zipf IDs, uniform gradients).

    python -m paper_2204_04179_b200.index_probe [--p 1000000] [--items 100000] [--s 1.1] [--d 768] [--iters 20]
    python -m paper_2204_04179_b200.index_probe --sweep [--iters 10]

Prints one JSON line with milliseconds and achieved GB/s (algorithmic bytes / time) per kernel.
"""
import argparse
import json
import statistics

import torch

from paper_2204_04179_b200 import binding, synth


def run_cell(P, N, s, d, iters=20, dev="cuda:0", seed=1):
    cfg = binding.GramConfig(); cfg.n_items = N; cfg.P_max = P; cfg.d_max = d; cfg.d = d
    g = binding.Gram(cfg)
    ids = torch.from_numpy(synth.zipf_ids(seed, N, s, P)).to(dev)
    cap = min(P, N)
    unique = torch.empty(cap, dtype=torch.int32, device=dev); inverse = torch.empty(P, dtype=torch.int32, device=dev)
    perm = torch.empty(P, dtype=torch.int32, device=dev); seg = torch.empty(cap + 1, dtype=torch.int32, device=dev)
    nu = torch.zeros(1, dtype=torch.int32, device=dev)
    g.dedup(ids, N, unique, inverse, perm, seg, nu); g.sync()
    U = int(nu.item())
    H = torch.randn(U, d, device=dev); E = torch.empty(P, d, device=dev)
    dE = torch.empty(P, d, device=dev).uniform_(-1, 1); G = torch.empty(U, d, device=dev)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than the 126 MB L2

    def timeit(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(iters):
            flush.zero_()                                                   # evict the previous iteration's lines
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); torch.cuda.synchronize(); ts.append(a.elapsed_time(b))
        return statistics.median(ts)
    passes = (max(1, (N - 1).bit_length()) + 7) // 8
    out = {"P": P, "n_items": N, "zipf_s": s, "d": d, "U": U,
           "working_set_MB": (4.0 * P * d + 4.0 * U * d) / 1e6}
    for name, fn, nbytes in (
            ("dedup", lambda: g.dedup(ids, N, unique, inverse, perm, seg, nu), (16 * passes + 20) * P + 8 * U),
            ("gather", lambda: g.gather(H, inverse, E), 4 * P * d + 4 * U * d + 4 * P),
            ("accumulate", lambda: g.accumulate(dE, perm, seg, U, G), 4 * P * d + 4 * U * d + 4 * P + 4 * (U + 1))):
        ms = timeit(fn)
        out[name] = {"ms": ms, "GB/s": nbytes / ms / 1e6}
    g.close()
    return out


def sweep(budget_gb: float = 12.0, iters: int = 10):
    """The kernel sweep: P in 1e4..1e7, item pool 1e3..1e6, Zipf s in {0.8, 1.1, 1.5}, d in {256, 768, 1024}.
    Cells whose gradient buffer (4*P*d bytes) exceeds the budget are listed as pruned, not run."""
    import torch
    for P in (10**4, 10**5, 10**6, 10**7):
        for d in (256, 768, 1024):
            if 4.0 * P * d > budget_gb * 1e9:
                print(json.dumps({"P": P, "d": d, "pruned": f"4*P*d = {4.0 * P * d / 1e9:.1f} GB exceeds the {budget_gb:.0f} GB per-buffer budget"}), flush=True)
                continue
            for N in (10**3, 10**4, 10**5, 10**6):
                for s in (0.8, 1.1, 1.5):
                    r = run_cell(P, N, s, d, iters)
                    r["l2_resident"] = r["working_set_MB"] < 126.0
                    print(json.dumps(r), flush=True)
                    torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--p", type=int, default=1_000_000)
    ap.add_argument("--items", type=int, default=100_000)
    ap.add_argument("--s", type=float, default=1.1)
    ap.add_argument("--d", type=int, default=768)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--sweep", action="store_true", help="run the whole grid (one JSON line per cell)")
    a = ap.parse_args()
    if a.sweep:
        sweep(iters=a.iters)
    else:
        print(json.dumps(run_cell(a.p, a.items, a.s, a.d, a.iters)))


if __name__ == "__main__":
    main()
