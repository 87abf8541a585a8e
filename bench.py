#!/usr/bin/env python
"""Benchmark of the GRAM training step (Single-step GRAM on the knowledge-tracing-shaped workload).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload kt|nr|tiny|kt_multistep|kt_6l|nr_additive]

A step is one pass of the whole path (dedup, encode unique items, gather, task module forward/backward,
accumulate, encoder backward) over one batch of seeded synthetic histories.  Prints ONE JSON line.
With --impl reference the CPU oracle (end-to-end training, one encoder call per interaction) is timed
instead, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "interactions/sec per GRAM train step on 1 B200; accumulate/gather GB/s vs HBM peak"
UNIT = "interactions/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops=p["bf16_tflops_sustained"], tflops_burst=p["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, tflops=1400.0, tflops_burst=1590.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                                          "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


def gemm_traffic_per_row():
    """DRAM bytes per token row of the forward qkv product from the committed ncu summary; None when gemm.cu has
    changed since the counters were taken."""
    import hashlib
    prof = os.path.join(ROOT, "profiles", "gemm_tc2_fwd_qkv_shape.md")
    src = os.path.join(ROOT, "paper_2204_04179_b200", "csrc", "gemm.cu")
    if not (os.path.exists(prof) and os.path.exists(src)):
        return None
    kv = {}
    for line in open(prof):
        if ":" in line and line.split(":")[0] in ("gemm_cu_sha256", "dram_bytes_per_row"):
            kv[line.split(":")[0]] = line.split(":", 1)[1].strip()
    if kv.get("gemm_cu_sha256") != hashlib.sha256(open(src, "rb").read()).hexdigest():
        return None
    return float(kv["dram_bytes_per_row"])


def oracle_sample(shape, ce, tk, toks, ids, lab, n_pos):
    """The oracle, as it stands, on the first n_pos positions of the first history: interactions/s."""
    import torch
    from oracle import gram_oracle as orc
    sub = shape.replace(B=1, L=n_pos)
    tk_sub = dict(tk)
    tk_sub["pos"] = tk["pos"][:n_pos] if "pos" in tk else None
    if tk_sub["pos"] is None:
        del tk_sub["pos"]
    t0 = time.time()
    orc.e2e_step(sub, ce, tk_sub, toks, ids[:1, :n_pos], lab[:1, :n_pos])
    dt = time.time() - t0
    return n_pos / dt, dt, torch.get_num_threads()


def bounded_sample_size(shape):
    if shape.name == "tiny":
        return shape.L
    return min(shape.L, 48 if shape.task == "kt" else shape.L)


def run_reference(args, shape):
    from paper_2204_04179_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ce = synth.encoder_params(shape, args.seed)
    tk = synth.task_params(shape, args.seed)
    toks = synth.item_tokens(args.seed, shape.n_items, shape.l_t, shape.vocab)
    if args.var_len:
        toks = synth.ragged(toks, synth.item_lengths(args.seed, shape.n_items, shape.l_t, shortest=min(4, shape.l_t)))
    n_pos = min(bounded_sample_size(shape), 12 if shape.name != "tiny" else shape.L)
    times, cores = [], 0
    for k in range(args.warmup + args.steps):
        ids, lab = synth.batch(shape, args.seed, step=k)
        v, dt, cores = oracle_sample(shape, ce, tk, toks, ids, lab, n_pos)
        if k >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = n_pos * len(times) / total
    sample = f"end-to-end oracle (float64, one encoder call per interaction) on the first {n_pos} positions of one history per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": shape.name, "B": 1, "L": n_pos, "n_items": shape.n_items, "note": "bounded sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def stack_flops(tokens, n_layers, d, d_ff, seq, attn_only=False):
    """Forward flops of n_layers transformer layers over `tokens` rows in sequences of `seq` rows: the four projections,
    the feed-forward products (2 flops per multiply-add) and the two attention products."""
    per_layer = 2.0 * 4 * d * d + (0.0 if attn_only else 2.0 * 2 * d * d_ff) + 4.0 * seq * d
    return tokens * n_layers * per_layer


def stage_fractions(shape, stage_ms, U, peaks):
    """Algorithmic work of each stage of a Single-step step (fixed-length texts) over its device time, against the
    roofline that bounds it: HBM bytes for dedup, gather and accumulate, bf16 tensor flops for the three model stages.
    With token-0 pooling the row-wise part of the last encoder layer is needed for one row per item only; the flops
    counted are those the method needs, not the ones a plain implementation would spend."""
    P, d, N = shape.B * shape.L, shape.d, shape.n_items
    passes = (max(1, (N - 1).bit_length()) + 7) // 8
    T = U * shape.l_t
    enc = stack_flops(T, shape.n_layers, d, shape.d_ff, shape.l_t)
    if shape.pooling == "cls" and shape.n_layers > 0:          # output projection + feed-forward of the last layer: U rows, not T
        enc -= (T - U) * (2.0 * d * d + 2.0 * 2 * d * shape.d_ff)
    if shape.task == "kt":
        task = 3.0 * stack_flops(P, shape.task_layers, d, shape.task_d_ff, shape.L / 2.0, shape.task_attn_only)   # causal: half the scores
    else:
        task = 3.0 * 2.0 * P * d * shape.d_a
    work = {"ms_dedup": ((16 * passes + 20) * P + 8 * U, "hbm"),
            "ms_encode": (enc, "tensor"),
            "ms_gather": (4.0 * P * d + 4.0 * U * d + 4 * P, "hbm"),
            "ms_task": (task, "tensor"),
            "ms_accumulate": (4.0 * P * d + 4.0 * U * d + 4 * P + 4 * (U + 1), "hbm"),
            "ms_backward": (2.0 * enc, "tensor")}
    out = {}
    for k, (w, bound) in work.items():
        ms = stage_ms[k]
        if ms <= 0:
            continue
        rate = w / (ms / 1e3)
        if bound == "hbm":
            out[k[3:]] = {"bound": "hbm", "GB/s": rate / 1e9, "frac": rate / (peaks["hbm_gbs"] * 1e9)}
        elif shape.dtype == "bf16":
            out[k[3:]] = {"bound": "tensor", "TFLOP/s": rate / 1e12, "frac": rate / (peaks["tflops"] * 1e12)}
        else:       # fp32 contexts run on the plain ALUs: 148 SMs x 128 fused multiply-adds per clock x 1.965 GHz
            out[k[3:]] = {"bound": "alu", "TFLOP/s": rate / 1e12, "frac": rate / (148 * 128 * 2 * 1.965e9)}
    out["note"] = ("algorithmic bytes or flops of the stage / its device time; dedup, gather and accumulate move tens of MB here "
                   "(L2-resident, launch-latency scale): their HBM fractions are taken on the larger cell under hbm_kernels")
    return out


def kernel_sweep_cell(binding, synth, torch, dev, peaks):
    """dedup / gather / accumulate alone on one sweep cell larger than L2 (P=1e6, N=1e5, Zipf 1.1, d=768)."""
    P, N, s, d = 1_000_000, 100_000, 1.1, 768
    cfg = binding.GramConfig(); cfg.n_items = N; cfg.P_max = P; cfg.d_max = d; cfg.d = d
    g = binding.Gram(cfg)
    ids = torch.from_numpy(synth.zipf_ids(1, N, s, P)).to(dev)
    cap = min(P, N)
    unique = torch.empty(cap, dtype=torch.int32, device=dev); inverse = torch.empty(P, dtype=torch.int32, device=dev)
    perm = torch.empty(P, dtype=torch.int32, device=dev); seg = torch.empty(cap + 1, dtype=torch.int32, device=dev)
    nu = torch.zeros(1, dtype=torch.int32, device=dev)
    g.dedup(ids, N, unique, inverse, perm, seg, nu); g.sync()
    U = int(nu.item())
    H = torch.randn(U, d, device=dev); E = torch.empty(P, d, device=dev)
    dE = torch.randn(P, d, device=dev); G = torch.empty(U, d, device=dev)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than the 126 MB L2

    def timeit(fn, n=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(n):
            flush.zero_()                                                   # evict the previous iteration's lines
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); torch.cuda.synchronize(); ts.append(a.elapsed_time(b))
        return statistics.median(ts)
    passes = (max(1, (N - 1).bit_length()) + 7) // 8
    out = {}
    for name, fn, nbytes in (
            ("dedup", lambda: g.dedup(ids, N, unique, inverse, perm, seg, nu), (16 * passes + 20) * P + 8 * U),
            ("gather_f32", lambda: g.gather(H, inverse, E), 4 * P * d + 4 * U * d + 4 * P),
            ("accumulate", lambda: g.accumulate(dE, perm, seg, U, G), 4 * P * d + 4 * U * d + 4 * P + 4 * (U + 1))):
        ms = timeit(fn)
        out[name] = {"ms": ms, "GB/s": nbytes / ms / 1e6, "frac_of_" + peaks["source"] + "_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"]}
    out["cell"] = {"P": P, "n_items": N, "zipf_s": s, "d": d, "U": U, "l2": "flushed between timed iterations"}
    del H, E, dE, G
    # the optimiser's update on a parameter vector the size of the BERT-base-shaped encoder (with its bf16 copy)
    n = 108_891_648
    w = torch.randn(n, device=dev) * 0.02; gr = torch.randn(n, device=dev) * 1e-3
    m = torch.zeros(n, device=dev); v = torch.zeros(n, device=dev); wb = torch.empty(n, dtype=torch.bfloat16, device=dev)
    step = [0]

    def adam():
        step[0] += 1
        g.adam_update(w, gr, m, v, step[0], 1e-4, w_bf16=wb)
    ms = timeit(adam)
    nbytes = 30 * n
    out["adam_update"] = {"ms": ms, "GB/s": nbytes / ms / 1e6, "frac_of_" + peaks["source"] + "_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"],
                          "params": n}
    g.close()
    return out


def run_gram(args, shape):
    import torch
    from paper_2204_04179_b200 import binding, synth
    from paper_2204_04179_b200 import dist as gdist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    peaks = measured_peaks()

    ce = synth.encoder_params(shape, args.seed)
    tk = synth.task_params(shape, args.seed)
    toks = synth.item_tokens(args.seed, shape.n_items, shape.l_t, shape.vocab)
    over = {}
    if args.micro_batch:
        over["ce_micro_batch"] = args.micro_batch
    multistep = shape.K > 1
    if multistep:                      # whole windows only: K-1 light steps and one step with the encoder pass
        over["lr_task"] = 1e-3
        if args.multistep_variant == "pseudo_target":
            over["multistep_variant"] = binding.GRAM_MULTI_PSEUDO_TARGET
        args.warmup = max(shape.K, -(-args.warmup // shape.K) * shape.K)
        args.steps = max(shape.K, -(-args.steps // shape.K) * shape.K)
    cfg = binding.config_from_shape(shape, **over)
    g = binding.Gram(cfg)
    g.set_params(binding.GRAM_MODULE_CE, synth.flatten(ce))
    g.set_params(binding.GRAM_MODULE_TASK, synth.flatten(tk))
    g.set_item_tokens(toks)
    lengths = None
    if args.var_len:                   # texts of 4 .. l_t tokens, uniform: the encoder then works on packed rows
        lengths = synth.item_lengths(args.seed, shape.n_items, shape.l_t, shortest=min(4, shape.l_t))
        g.set_item_lengths(lengths)
    P = shape.B * shape.L
    n_total = args.warmup + args.steps
    # every rank draws its own batches (weak scaling: per-GPU work is fixed, histories are independent)
    batches = [synth.batch(shape, gdist.rank_seed(args.seed, rank), step=k) for k in range(n_total)]
    dev_batches = [(torch.from_numpy(i).to(dev), torch.from_numpy(l).to(dev)) for i, l in batches]
    pinned = [(torch.from_numpy(i).pin_memory(), torch.from_numpy(l).pin_memory()) for i, l in batches]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return gdist.max_over_ranks(ms, dist, dev)

    # ---- device-resident inputs ----
    if multistep:
        g.cache_fill()                 # encodings of every item with the initial parameters (untimed set-up)
    for k in range(args.warmup):
        g.step(dev_batches[k][0], dev_batches[k][1], shape.B)
    g.profile(True)
    launches0 = g.launch_count()
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    reports = []
    for k in range(args.warmup, n_total):
        reports.append(g.step(dev_batches[k][0], dev_batches[k][1], shape.B))
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    launches = g.launch_count() - launches0
    kinds = g.profile_read()
    sites = g.profile_dump()
    g.profile(False)

    # ---- end to end: host buffers through gram_step_host (copies inside the timed region) ----
    for k in range(min(args.warmup, 1)):
        g.step_host(pinned[k][0].numpy(), pinned[k][1].numpy(), shape.B)
    barrier()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for k in range(args.warmup, n_total):
        g.step_host(pinned[k][0].numpy(), pinned[k][1].numpy(), shape.B)
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1))

    if rank != 0:
        g.close()
        return
    value = world * P * args.steps / (ms_total / 1e3)
    e2e_value = world * P * args.steps / (ms_e2e / 1e3)
    gm = kinds["gemm"]
    achieved = gm["work"] / (gm["ms"] / 1e3) / 1e12 if gm["ms"] > 0 else 0.0
    roofline = {"kernel": "gemm_tc_kernel (bf16 tcgen05, fp32 accumulate)" if shape.dtype == "bf16" else "gemm_f32_kernel",
                "bound": "tensor" if shape.dtype == "bf16" else "alu",
                "achieved": achieved, "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"],
                "peak_source": peaks["source"] + " bf16_tflops_sustained", "traffic": None,
                "traffic_note": "DRAM bytes of one fwd_qkv launch (tokens x 2304 x 768), scaled by rows from the ncu capture "
                                "in profiles/gemm_tc2_fwd_qkv_shape.md; null when gemm.cu changed since that capture",
                "launches": gm["launches"], "avg_launch_ms": gm["ms"] / max(1, gm["launches"]),
                "share_of_step": gm["ms"] / (ms_total if ms_total > 0 else 1)}
    per_row = gemm_traffic_per_row()
    if per_row is not None and shape.dtype == "bf16" and lengths is None:      # rows per launch are known only for fixed-length texts
        roofline["traffic"] = per_row * statistics.mean(r.n_unique for r in reports) * shape.l_t
    stage_ms = {k: statistics.mean(getattr(r, k) for r in reports)
                for k in ("ms_dedup", "ms_encode", "ms_gather", "ms_task", "ms_accumulate", "ms_backward", "ms_total")}
    stage_roofline = stage_fractions(shape, stage_ms, statistics.mean(r.n_unique for r in reports), peaks) \
        if (not multistep and lengths is None) else None
    per_kind = {}
    for name, v in kinds.items():
        if v["launches"] == 0:
            continue
        rate = v["work"] / (v["ms"] / 1e3) if v["ms"] > 0 else 0.0
        is_flops = name in ("gemm", "attention")
        per_kind[name] = {"ms_per_step": v["ms"] / args.steps, "launches_per_step": v["launches"] / args.steps,
                          ("TFLOP/s" if is_flops else "GB/s"): rate / (1e12 if is_flops else 1e9),
                          "frac": rate / ((peaks["tflops"] * 1e12) if is_flops else (peaks["hbm_gbs"] * 1e9))}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": shape.dtype, "data": "synthetic",
        "config": {"workload": shape.name, "B": shape.B, "L": shape.L, "n_items": shape.n_items, "l_t": shape.l_t,
                   "encoder": f"{shape.n_layers}x{shape.d} ({shape.n_heads} heads, ffn {shape.d_ff}), {shape.pooling} pooling",
                   "task": shape.task, "zipf_s": shape.zipf_s, "unique_items_per_step": statistics.mean(r.n_unique for r in reports),
                   "boost_ratio_R": statistics.mean(r.boost_ratio for r in reports), "ce_micro_batch": int(cfg.ce_micro_batch),
                   "l2": "working set (activations of >1e5 tokens) far larger than L2; no flush needed",
                   "text_lengths": ("uniform 4..l_t, mean %.1f tokens" % float(lengths.mean())) if lengths is not None else "all l_t",
                   "parallelism": f"replicas x{world}" if world > 1 else "1 GPU"},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 8 * P, "d2h_bytes_per_step": 12,
                "ms_per_step": ms_e2e / args.steps},
        "roofline": roofline, "stage_ms": stage_ms, "stage_roofline": stage_roofline, "kernel_kinds": per_kind,
        "call_sites": {t: {"ms_per_step": v["ms"] / args.steps, "launches_per_step": v["launches"] / args.steps,
                           ("TFLOP/s" if v["kind"] in ("gemm", "attention") else "GB/s"):
                               (v["work"] / (v["ms"] / 1e3) / (1e12 if v["kind"] in ("gemm", "attention") else 1e9)) if v["ms"] > 0 else 0.0}
                       for t, v in sites.items()},
    }
    g.close()
    if world == 1:
        del dev_batches
        torch.cuda.empty_cache()
        try:
            line["hbm_kernels"] = kernel_sweep_cell(binding, synth, torch, dev, peaks)
        except Exception as ex:          # the sweep cell is extra information, never a reason to lose the line
            line["hbm_kernels"] = {"error": repr(ex)}
        n_pos = bounded_sample_size(shape)
        toks_o = synth.ragged(toks, lengths) if lengths is not None else toks
        v, dt, cores = oracle_sample(shape, ce, tk, toks_o, batches[0][0], batches[0][1], n_pos)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"end-to-end oracle (float64, one encoder call per interaction) on the first {n_pos} "
                                          f"positions of one history of the same workload, {dt:.1f} s; linear in interactions"}
    if multistep:
        line["multistep"] = {"K": shape.K, "windows_timed": args.steps // shape.K, "variant": args.multistep_variant,
                             "per_step": [{"k": i % shape.K, "ms": r.ms_total, "touched": r.n_touched,
                                           "encoder_pass": r.encoder_pass, "n_encoded": r.n_encoded} for i, r in enumerate(reports)]}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="gram", choices=["gram", "reference"])
    ap.add_argument("--workload", default="kt", choices=["kt", "nr", "tiny", "kt_multistep", "kt_6l", "nr_additive"])
    ap.add_argument("--micro-batch", type=int, default=0, help="items per encoder pass (0: the workload's default)")
    ap.add_argument("--multistep-variant", default="table", choices=["table", "pseudo_target"],
                    help="kt_multistep: separate gradient table with unchanged cached encodings, or pseudo-targets (Section 4.3)")
    ap.add_argument("--var-len", action="store_true", help="item texts of different lengths (uniform 4..l_t) instead of all l_t")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    from paper_2204_04179_b200 import synth
    shape = synth.config(args.workload)
    if args.workload in ("kt", "nr", "kt_multistep", "kt_6l", "nr_additive") and not args.micro_batch:
        args.micro_batch = 0 if args.workload in ("nr", "nr_additive") else 5120
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        run_gram(args, shape)


if __name__ == "__main__":
    main()
