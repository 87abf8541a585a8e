#!/usr/bin/env python
"""Benchmark of the GRAM training step (Single-step GRAM on the knowledge-tracing-shaped workload).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload kt|nr|tiny|kt_multistep|kt_6l|nr_additive|nr_mhsa|sweep|gemm_sites]

A step is one pass of the whole path (dedup, encode unique items, gather, task module forward/backward,
accumulate, encoder backward, optimiser update) over one batch of seeded synthetic histories.  Prints ONE JSON line.
With --impl reference the CPU oracle (end-to-end training, one encoder call per interaction) is timed
instead, on a bounded sample of the same workload.

Other modes (each prints JSON lines of its own, none of them is the contract's line):
  --workload sweep       dedup / gather / accumulate alone over the grid P x item pool x Zipf s x d (--cell P,N,s,d: one cell)
  --workload gemm_sites  every matrix-product call site of the encoder at --rows token rows, with its epilogue, the same
                         shape through torch.matmul beside it as a measuring stick (--site NAME: one site, for profilers)
  --layers / --batch / --items cut a model workload down to a small case for profilers.
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
MODEL_WORKLOADS = ("kt", "nr", "tiny", "kt_multistep", "kt_6l", "nr_additive", "nr_mhsa")


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
    prof = os.path.join(ROOT, "profiles", "gemm_call_sites_65536_rows.md")
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
    if "pos" in tk:
        tk_sub["pos"] = tk["pos"][:n_pos]
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
        if ms <= 0 or (k == "ms_gather" and shape.task == "kt"):     # the KT module gathers in its first load: no stage of its own
            continue
        rate = w / (ms / 1e3)
        if bound == "hbm":
            out[k[3:]] = {"bound": "hbm", "GB/s": rate / 1e9, "frac": rate / (peaks["hbm_gbs"] * 1e9)}
        elif shape.dtype == "bf16":
            out[k[3:]] = {"bound": "tensor", "TFLOP/s": rate / 1e12, "frac": rate / (peaks["tflops"] * 1e12)}
        else:       # fp32 contexts run on the plain ALUs: 148 SMs x 128 fused multiply-adds per clock x 1.965 GHz
            out[k[3:]] = {"bound": "alu", "TFLOP/s": rate / 1e12, "frac": rate / (148 * 128 * 2 * 1.965e9)}
    out["note"] = ("algorithmic bytes or flops of the stage / its device time; dedup, gather and accumulate move tens of MB here "
                   "(L2-resident, launch-latency scale): their HBM fractions are taken on the larger cell under hbm_kernels; "
                   "with the KT task module the gather runs inside the module's first kernel (ms_gather is then ~0 and its "
                   "bytes are part of ms_task)")
    return out


# ---------------------------------------------------------------------------------------------------------------------
# index kernels alone (the accumulate / gather sweep)
# ---------------------------------------------------------------------------------------------------------------------

def index_cell(binding, synth, torch, dev, P, N, s, d, iters=20, seed=1, peaks=None):
    """dedup, gather and accumulate alone on one cell: seeded Zipf IDs, uniform gradients, L2 flushed between iterations."""
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
    out = {"cell": {"P": P, "n_items": N, "zipf_s": s, "d": d, "U": U, "working_set_MB": (4.0 * P * d + 4.0 * U * d) / 1e6,
                    "l2": "flushed between timed iterations"}}
    for name, fn, nbytes in (
            ("dedup", lambda: g.dedup(ids, N, unique, inverse, perm, seg, nu), (16 * passes + 20) * P + 8 * U),
            ("gather_f32", lambda: g.gather(H, inverse, E), 4 * P * d + 4 * U * d + 4 * P),
            ("accumulate", lambda: g.accumulate(dE, perm, seg, U, G), 4 * P * d + 4 * U * d + 4 * P + 4 * (U + 1))):
        ms = timeit(fn)
        out[name] = {"ms": ms, "GB/s": nbytes / ms / 1e6}
        if peaks:
            out[name]["frac_of_" + peaks["source"] + "_hbm"] = nbytes / ms / 1e6 / peaks["hbm_gbs"]
    g.close()
    return out


def adam_cell(binding, torch, dev, peaks):
    """The optimiser's update on a parameter vector the size of the BERT-base-shaped encoder (with its bf16 copy)."""
    cfg = binding.GramConfig(); cfg.n_items = 8; cfg.P_max = 8; cfg.d = 8
    g = binding.Gram(cfg)
    n = 108_891_648
    w = torch.randn(n, device=dev) * 0.02; gr = torch.randn(n, device=dev) * 1e-3
    m = torch.zeros(n, device=dev); v = torch.zeros(n, device=dev); wb = torch.empty(n, dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    ts = []
    for it in range(1, 24):
        flush.zero_()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record(); g.adam_update(w, gr, m, v, it, 1e-4, w_bf16=wb); b.record(); torch.cuda.synchronize()
        if it > 3:
            ts.append(a.elapsed_time(b))
    ms = statistics.median(ts)
    g.close()
    nbytes = 30 * n
    return {"ms": ms, "GB/s": nbytes / ms / 1e6, "frac_of_" + peaks["source"] + "_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"], "params": n}


def run_sweep(args):
    """The kernel sweep: P in 1e4..1e7, item pool 1e3..1e6, Zipf s in {0.8, 1.1, 1.5}, d in {256, 768, 1024}; one JSON
    line per cell.  A cell holds three P x d fp32 buffers (source rows, gathered rows, gradients); cells whose buffers
    would exceed --sweep-budget-gb each are listed as pruned, not run."""
    import torch
    from paper_2204_04179_b200 import binding, synth
    dev = "cuda:0"
    peaks = measured_peaks()
    if args.cell:
        P, N, s, d = args.cell.split(",")
        print(json.dumps(index_cell(binding, synth, torch, dev, int(float(P)), int(float(N)), float(s), int(d), args.iters, peaks=peaks)))
        return
    for P in (10**4, 10**5, 10**6, 10**7):
        for d in (256, 768, 1024):
            if 4.0 * P * d > args.sweep_budget_gb * 1e9:
                print(json.dumps({"P": P, "d": d, "pruned": f"4*P*d = {4.0 * P * d / 1e9:.1f} GB exceeds the "
                                  f"{args.sweep_budget_gb:.0f} GB per-buffer budget (--sweep-budget-gb)"}), flush=True)
                continue
            for N in (10**3, 10**4, 10**5, 10**6):
                for s in (0.8, 1.1, 1.5):
                    r = index_cell(binding, synth, torch, dev, P, N, s, d, args.iters, peaks=peaks)
                    r["cell"]["l2_resident"] = r["cell"]["working_set_MB"] < 126.0
                    print(json.dumps(r), flush=True)
                    torch.cuda.empty_cache()


# ---------------------------------------------------------------------------------------------------------------------
# the matrix products of one encoder layer, call site by call site
# ---------------------------------------------------------------------------------------------------------------------

def gemm_sites(d=768, d_ff=3072):
    """(name, layout, N, K, epilogue) of every matrix-product call site of a layer's forward and backward pass.
    Layouts: tn = A [M,K] B [N,K] (forward), nn = A [M,K] B [K,N] (input gradient), tt = A [K,M] B [K,N] (weight
    gradient: M and N are the weight's sides, K is the token count)."""
    return [("fwd_qkv", "tn", 3 * d, d, "bias"), ("fwd_attn_out", "tn", d, d, "res_ln"), ("fwd_ffn1", "tn", d_ff, d, "gelu"),
            ("fwd_ffn2", "tn", d, d_ff, "res_ln"), ("dx_ffn2_dgelu", "nn", d_ff, d, "dgelu"), ("dx_ffn1", "nn", d, d_ff, "res"),
            ("dx_attn_out", "nn", d, d, "plain"), ("dx_qkv", "nn", d, 3 * d, "res"),
            ("dw_ffn2", "tt", d, d_ff, "acc"), ("dw_ffn1", "tt", d_ff, d, "acc"), ("dw_attn_out", "tt", d, d, "acc"),
            ("dw_qkv", "tt", 3 * d, d, "acc")]


def run_gemm_sites(args):
    import torch
    from paper_2204_04179_b200 import binding
    dev = "cuda:0"
    peaks = measured_peaks()
    cfg = binding.GramConfig(); cfg.n_items = 8; cfg.P_max = 8; cfg.d = 8; cfg.d_ff = 4096
    g = binding.Gram(cfg)
    T = args.rows
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for name, layout, N, K, epi in gemm_sites():
        if args.site and name != args.site:
            continue
        bf = torch.bfloat16
        if layout == "tt":          # dW[N_w, K_w] += dY[T, N_w]^T X[T, K_w]
            M_, N_, K_ = N, K, T
            A = (torch.randn(T, N, device=dev) * 0.5).to(bf); Bm = (torch.randn(T, K, device=dev) * 0.5).to(bf)
            Cm = torch.zeros(N, K, device=dev)
            run = lambda: g.gemm_bf16(A, 0, Bm, 0, Cm, None, 1, M_, N_, K_)
            stick = lambda: torch.matmul(A.T, Bm)
        else:
            M_, N_, K_ = T, N, K
            A = (torch.randn(T, K, device=dev) * 0.5).to(bf)
            Bm = (torch.randn(N, K, device=dev) * 0.05).to(bf) if layout == "tn" else (torch.randn(K, N, device=dev) * 0.05).to(bf)
            b_k = 1 if layout == "tn" else 0
            kw = {}
            c_f32 = epi in ("res", "res_ln")
            Cm = torch.empty(T, N, device=dev, dtype=torch.float32 if c_f32 else bf)
            if epi in ("bias", "gelu", "res_ln"):
                kw["bias"] = torch.randn(N, device=dev) * 0.1
            if epi == "gelu":
                kw["gelu"] = True; kw["gelu_grad_out"] = torch.empty(T, N, device=dev, dtype=bf)
            if epi == "dgelu":
                kw["gelu_grad_in"] = torch.rand(T, N, device=dev).to(bf)
            if epi in ("res", "res_ln"):
                kw["res"] = torch.randn(T, N, device=dev)
            if epi == "res_ln":
                kw["res_ln"] = (torch.randn(T, device=dev) * 0.1, torch.rand(T, device=dev) + 0.5, torch.rand(N, device=dev) + 0.5,
                                torch.randn(N, device=dev) * 0.1)
            run = (lambda A=A, Bm=Bm, Cm=Cm, b_k=b_k, kw=kw: g.gemm_bf16_epilogue(A, 1, Bm, b_k, Cm, M_, N_, K_, **kw))
            stick = (lambda: torch.matmul(A, Bm.T)) if layout == "tn" else (lambda: torch.matmul(A, Bm))

        def timeit(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            ts = []
            for _ in range(args.iters):
                flush.zero_()
                a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record(); torch.cuda.synchronize(); ts.append(a.elapsed_time(b))
            return statistics.median(ts)
        flops = 2.0 * M_ * N_ * K_
        ms = timeit(run)
        line = {"site": name, "layout": layout, "M": M_, "N": N_, "K": K_, "epilogue": epi, "ms": ms, "TFLOP/s": flops / ms / 1e9,
                "frac_of_" + peaks["source"] + "_sustained": flops / ms / 1e9 / peaks["tflops"]}
        if not args.site:            # the measuring stick: the library product on the same shape, without the epilogue
            ms_t = timeit(stick)
            line["torch_matmul_plain"] = {"ms": ms_t, "TFLOP/s": flops / ms_t / 1e9}
        print(json.dumps(line), flush=True)
        del A, Bm, Cm
        torch.cuda.empty_cache()
    g.close()


# ---------------------------------------------------------------------------------------------------------------------
# the training step
# ---------------------------------------------------------------------------------------------------------------------

class StepRun:
    """One library context on one workload with its seeded batches resident on the device and in pinned host memory."""

    def __init__(self, args, shape, rank, dev, n_total, multistep_variant="table"):
        import torch
        from paper_2204_04179_b200 import binding, synth
        from paper_2204_04179_b200 import dist as gdist
        self.shape, self.dev = shape, dev
        self.ce = synth.encoder_params(shape, args.seed)
        self.tk = synth.task_params(shape, args.seed)
        self.toks = synth.item_tokens(args.seed, shape.n_items, shape.l_t, shape.vocab)
        over = {}
        if shape.name not in ("tiny",) and shape.task == "kt":
            over["ce_micro_batch"] = args.micro_batch if args.micro_batch else 5120
        elif args.micro_batch:
            over["ce_micro_batch"] = args.micro_batch
        # a full training step: Adam under the Noam scheme at the paper's rate (Appendix D) for both modules
        over.update(optimizer=binding.GRAM_OPT_ADAM, lr_task=1e-4, lr_ce=1e-4, noam_warmup=4000)
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        if self.world > 1:
            over["defer_update"] = 1       # gradients are averaged over the replicas before the update
        self.multistep = shape.K > 1
        if self.multistep and multistep_variant == "pseudo_target":
            over["multistep_variant"] = binding.GRAM_MULTI_PSEUDO_TARGET
        self.cfg = binding.config_from_shape(shape, **over)
        self.g = binding.Gram(self.cfg)
        self.g.set_params(binding.GRAM_MODULE_CE, synth.flatten(self.ce))
        self.g.set_params(binding.GRAM_MODULE_TASK, synth.flatten(self.tk))
        self.g.set_item_tokens(self.toks)
        self.lengths = None
        if args.var_len:                   # texts of 4 .. l_t tokens, uniform: the encoder then works on packed rows
            self.lengths = synth.item_lengths(args.seed, shape.n_items, shape.l_t, shortest=min(4, shape.l_t))
            self.g.set_item_lengths(self.lengths)
        # every rank draws its own batches (weak scaling: per-GPU work is fixed, histories are independent)
        self.batches = [synth.batch(shape, gdist.rank_seed(args.seed, rank), step=k) for k in range(n_total)]
        self.dev_batches = [(torch.from_numpy(i).to(dev), torch.from_numpy(l).to(dev)) for i, l in self.batches]
        self.pinned = [(torch.from_numpy(i).pin_memory(), torch.from_numpy(l).pin_memory()) for i, l in self.batches]
        self.n_pred = [gdist.n_predictions(shape, l) for _, l in self.batches]
        if self.multistep:
            self.g.cache_fill()            # encodings of every item with the initial parameters (untimed set-up)

    def step(self, k, dist=None, host=False):
        from paper_2204_04179_b200 import binding
        from paper_2204_04179_b200 import dist as gdist
        if host:
            rep = self.g.step_host(self.pinned[k][0].numpy(), self.pinned[k][1].numpy(), self.shape.B)
        else:
            rep = self.g.step(self.dev_batches[k][0], self.dev_batches[k][1], self.shape.B)
        if self.world > 1:                 # data-parallel replicas: one gradient all-reduce per update, then the update
            if rep.encoder_pass:
                gdist.allreduce_grads(self.g, self.n_pred[k], dist)
                self.g.optimizer_step(binding.GRAM_MODULE_CE)
            else:
                import torch
                ptr, n = self.g.grads_device(binding.GRAM_MODULE_TASK)
                gdist.allreduce_weighted_mean([torch.as_tensor(gdist._DeviceBuffer(ptr, n), device="cuda")], self.n_pred[k], dist)
            self.g.optimizer_step(binding.GRAM_MODULE_TASK)
        return rep

    def close(self):
        self.g.close()
        self.dev_batches = None


def timed_pass(run, first, n, barrier, dist, host=False):
    """n steps from batch `first`, bracketed by a barrier + synchronize on both sides; CUDA events on the current stream."""
    import torch
    barrier()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    reps = [run.step(k, dist, host) for k in range(first, first + n)]
    e1.record()
    barrier()
    return e0.elapsed_time(e1), reps


def short_run(args, name, rank, dev, barrier, dist, world, K=None, steps=5, warmup=3):
    """A short un-instrumented run of another workload, for the record: throughput, step time, unique / touched items, stages."""
    from paper_2204_04179_b200 import synth
    shape = synth.config(name)
    if K is not None:
        shape = shape.replace(K=K)
    if shape.K > 1:
        warmup, steps = shape.K, shape.K            # one window to warm up, one timed
    run = StepRun(args, shape, rank, dev, warmup + steps)
    for k in range(warmup):
        run.step(k, dist)
    ms, reps = timed_pass(run, warmup, steps, barrier, dist)
    P = shape.B * shape.L
    out = {"workload": shape.name, "K": shape.K, "steps": steps, "warmup": warmup, "ms_per_step": ms / steps,
           "value": world * P * steps / (ms / 1e3), "unit": UNIT, "P": P,
           "unique_items_per_step": statistics.mean(r.n_unique for r in reps)}
    if shape.K > 1:
        out["touched_at_window_end"] = reps[-1].n_touched
        out["n_encoded"] = reps[-1].n_encoded
        out["ms_light_step"] = statistics.mean(r.ms_total for r in reps[:-1]) if len(reps) > 1 else None
        out["ms_encoder_step"] = reps[-1].ms_total
        out["touched_per_step"] = [r.n_touched for r in reps]
    else:
        out["stage_ms"] = {k: statistics.mean(getattr(r, k) for r in reps)
                           for k in ("ms_dedup", "ms_encode", "ms_gather", "ms_task", "ms_accumulate", "ms_backward", "ms_total")}
    run.close()
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
    multistep = shape.K > 1
    if multistep:                      # whole windows only: K-1 light steps and one step with the encoder pass
        args.warmup = max(shape.K, -(-args.warmup // shape.K) * shape.K)
        args.steps = max(shape.K, -(-args.steps // shape.K) * shape.K)
    n_total = args.warmup + args.steps
    run = StepRun(args, shape, rank, dev, n_total, args.multistep_variant)
    g, cfg, lengths = run.g, run.cfg, run.lengths
    P = shape.B * shape.L

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return gdist.max_over_ranks(ms, dist, dev)

    for k in range(args.warmup):
        run.step(k, dist)
    # ---- pass 1: device-resident inputs, nothing instrumented: the headline value ----
    launches0 = g.launch_count()
    sampler = ClockSampler(local)
    sampler.start()
    ms_total, reports = timed_pass(run, args.warmup, args.steps, barrier, dist)
    clocks = sampler.stop()
    ms_total = max_over_ranks(ms_total)
    launches = g.launch_count() - launches0
    # ---- pass 2: end to end, host buffers through gram_step_host (copies inside the timed region) ----
    ms_e2e, _ = timed_pass(run, args.warmup, args.steps, barrier, dist, host=True)
    ms_e2e = max_over_ranks(ms_e2e)
    # ---- pass 3: the same steps with every kernel group bracketed by events: the breakdown (never the headline) ----
    g.profile(True)
    ms_prof, prof_reports = timed_pass(run, args.warmup, args.steps, barrier, dist)
    kinds = g.profile_read()
    sites = g.profile_dump()
    g.profile(False)
    light_sites = None
    if multistep and shape.K > 1:
        # one more window, with the K-1 steps that run no encoder pass instrumented on their own: where a light step's time goes
        g.profile(True)
        for k in range(args.warmup, args.warmup + shape.K - 1):
            run.step(k, dist)
        light_sites = g.profile_dump()
        g.profile(False)
        run.step(args.warmup + shape.K - 1, dist)

    if rank != 0:
        run.close()
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    value = world * P * args.steps / (ms_total / 1e3)
    e2e_value = world * P * args.steps / (ms_e2e / 1e3)
    gm = kinds["gemm"]
    achieved = gm["work"] / (gm["ms"] / 1e3) / 1e12 if gm["ms"] > 0 else 0.0
    roofline = {"kernel": "gemm_tc2_kernel (bf16 tcgen05 on CTA pairs, fp32 accumulate in tensor memory; gemm_tc_kernel for small products)"
                          if shape.dtype == "bf16" else "gemm_f32_kernel",
                "bound": "tensor" if shape.dtype == "bf16" else "alu",
                "achieved": achieved, "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"],
                "peak_source": peaks["source"] + " bf16_tflops_sustained", "traffic": None,
                "traffic_note": "DRAM bytes of one fwd_qkv launch (tokens x 2304 x 768), scaled by rows from an ncu capture of the "
                                "same kernel on 65536 rows; null when gemm.cu has changed since that capture",
                "launches": gm["launches"], "avg_launch_ms": gm["ms"] / max(1, gm["launches"]),
                "share_of_step": gm["ms"] / (ms_prof if ms_prof > 0 else 1),
                "timed_in": "the instrumented pass (CUDA events around each launch on its stream); value and ms_per_step come from the un-instrumented pass"}
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
                   "optimizer": "Adam + Noam (rate 1e-4, warm-up 4000) on both modules, inside the step",
                   "l2": "working set (activations of >1e5 tokens) far larger than L2; no flush needed",
                   "text_lengths": ("uniform 4..l_t, mean %.1f tokens" % float(lengths.mean())) if lengths is not None else "all l_t",
                   "parallelism": (f"data-parallel replicas x{world}: one NCCL all-reduce of the parameter gradients per update "
                                   "(weighted by predictions), then the update") if world > 1 else "1 GPU"},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 8 * P, "d2h_bytes_per_step": 16,
                "ms_per_step": ms_e2e / args.steps},
        "ms_per_step_instrumented": ms_prof / args.steps,
        "roofline": roofline, "stage_ms": stage_ms, "stage_roofline": stage_roofline, "kernel_kinds": per_kind,
        "call_sites": {t: {"ms_per_step": v["ms"] / args.steps, "launches_per_step": v["launches"] / args.steps,
                           ("TFLOP/s" if v["kind"] in ("gemm", "attention") else "GB/s"):
                               (v["work"] / (v["ms"] / 1e3) / (1e12 if v["kind"] in ("gemm", "attention") else 1e9)) if v["ms"] > 0 else 0.0}
                       for t, v in sites.items()},
    }
    if multistep:
        line["multistep"] = {"K": shape.K, "windows_timed": args.steps // shape.K, "variant": args.multistep_variant,
                             "light_step_call_sites": {t: {"ms_per_step": v["ms"] / (shape.K - 1), "launches_per_step": v["launches"] / (shape.K - 1)}
                                                       for t, v in (light_sites or {}).items()},
                             "per_step": [{"k": i % shape.K, "ms": r.ms_total, "touched": r.n_touched,
                                           "encoder_pass": r.encoder_pass, "n_encoded": r.n_encoded} for i, r in enumerate(reports)]}
    batches0 = run.batches[0]
    ce, tk, toks = run.ce, run.tk, run.toks
    run.close()
    torch.cuda.empty_cache()
    if world == 1 and not args.no_others:
        # the other named workloads, briefly, so that one record covers them: news recommendation, Multi-step at K = 8, and
        # Multi-step as the accumulation latency K grows (Section 4.4 varies it from one step to whole epochs)
        others = {}
        try:
            if shape.name != "nr":
                others["nr"] = short_run(args, "nr", rank, dev, barrier, dist, world)
            ks = [shape.K] if multistep else []
            sweep = []
            for K in (2, 4, 8, 16, 32):
                if K in ks:
                    continue
                sweep.append(short_run(args, "kt_multistep", rank, dev, barrier, dist, world, K=K))
                torch.cuda.empty_cache()
            others["kt_multistep_K_sweep"] = sweep
            others["note"] = ("K = 1 is the Single-step line itself; each K: one window to warm up, one window timed, Adam on both "
                              "modules, bf16 cache, table variant")
        except Exception as ex:          # extra information, never a reason to lose the line
            others["error"] = repr(ex)
        line["other_workloads"] = others
        torch.cuda.empty_cache()
    if world == 1:
        try:
            hk = index_cell(binding, synth, torch, dev, 1_000_000, 100_000, 1.1, 768, 20, peaks=peaks)
            hk["adam_update"] = adam_cell(binding, torch, dev, peaks)
            line["hbm_kernels"] = hk
        except Exception as ex:
            line["hbm_kernels"] = {"error": repr(ex)}
        n_pos = bounded_sample_size(shape)
        toks_o = synth.ragged(toks, lengths) if lengths is not None else toks
        v, dt, cores = oracle_sample(shape, ce, tk, toks_o, batches0[0], batches0[1], n_pos)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"end-to-end oracle (float64, one encoder call per interaction) on the first {n_pos} "
                                          f"positions of one history of the same workload, {dt:.1f} s; linear in interactions"}
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="gram", choices=["gram", "reference"])
    ap.add_argument("--workload", default="kt", choices=list(MODEL_WORKLOADS) + ["sweep", "gemm_sites"])
    ap.add_argument("--micro-batch", type=int, default=0, help="items per encoder pass (0: the workload's default)")
    ap.add_argument("--multistep-variant", default="table", choices=["table", "pseudo_target"],
                    help="kt_multistep: separate gradient table with unchanged cached encodings, or pseudo-targets (Section 4.3)")
    ap.add_argument("--K", type=int, default=0, help="kt_multistep: steps per window (default 8)")
    ap.add_argument("--var-len", action="store_true", help="item texts of different lengths (uniform 4..l_t) instead of all l_t")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--layers", type=int, default=0, help="cut-down case: encoder layers")
    ap.add_argument("--batch", type=int, default=0, help="cut-down case: histories per batch")
    ap.add_argument("--items", type=int, default=0, help="cut-down case: item pool")
    ap.add_argument("--l-t", type=int, default=0, help="tokens per item text (a longer-text variant of the workload)")
    ap.add_argument("--cell", default="", help="sweep: one cell P,N,s,d")
    ap.add_argument("--sweep-budget-gb", type=float, default=45.0, help="sweep: largest P x d fp32 buffer that is still run")
    ap.add_argument("--rows", type=int, default=65536, help="gemm_sites: token rows")
    ap.add_argument("--site", default="", help="gemm_sites: one call site")
    ap.add_argument("--iters", type=int, default=10, help="sweep / gemm_sites: timed iterations per kernel")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    if args.workload == "sweep":
        return run_sweep(args)
    if args.workload == "gemm_sites":
        return run_gemm_sites(args)
    from paper_2204_04179_b200 import synth
    shape = synth.config(args.workload)
    if args.K and shape.K > 1:
        shape = shape.replace(K=args.K)
    if args.layers or args.batch or args.items or args.l_t:
        shape = shape.replace(n_layers=args.layers or shape.n_layers, B=args.batch or shape.B, n_items=args.items or shape.n_items,
                              l_t=args.l_t or shape.l_t)
        args.no_others = True
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        run_gram(args, shape)


if __name__ == "__main__":
    main()
