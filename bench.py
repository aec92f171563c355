#!/usr/bin/env python
"""Benchmark of the low-bit linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the 7B-class decoder linear stack (32 layers x
{q,k,v,o,gate,up,down}, per-matrix 2/3/4-bit codes with mean width 2.5,
blocks of 32 with fp16 scale+min) for M = 1 action decode: every packed weight
byte is streamed once, with the glue (RMS scale, SiLU*up, residual adds)
between the linears.  The headline metric is weight-stream GB/s.  The same
JSON line carries the prefill (M = 512) TFLOP/s of the same stack, the
standalone dequant GB/s, roofline fractions and the CPU oracle timed on the
host cores.  With N > 1 every rank runs an independent replica (the path does
not shard); value is the sum over ranks over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while a region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [s.strip() for s in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


def _timed(fn, steps, warmup, torch):
    """CUDA-event time of `steps` calls after `warmup` calls, in ms (total)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def reduce_max(values, dist, device):
    """Max over ranks of each entry (the slowest rank decides a multi-rank time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_gbs(world, packed_bytes_per_rank, ms_per_step):
    """Replicas only: every rank streams its own copy of the weights; the job's rate is the sum."""
    return world * packed_bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def oracle_layer_sample(which=("q", "k", "v", "o", "gate", "up", "down")):
    """Host-side inputs for the oracle timing: one 7B-shaped layer (or part of it)."""
    import numpy as np
    from oracle import aq_oracle as O
    from paper_2605_24011_b200 import synth
    shapes = [s for s in synth.llama7b_layer() if s[0] in which]
    bits = {"q": 2, "k": 2, "v": 3, "o": 3, "gate": 2, "up": 2, "down": 4}
    mats = []
    for i, (name, N, K) in enumerate(shapes):
        W = synth.weights(N, K, 77, i, outliers=True)
        d, m, q = O.quantize(W, bits[name])
        x = synth.activations(1, K, 77, i).astype(np.float16).astype(np.float64)
        mats.append((d, m, q, x, N * K * (bits[name] + 1) // 8))
    return mats


def time_oracle(mats, repeats=1):
    from oracle import aq_oracle as O
    t0 = time.perf_counter()
    for _ in range(repeats):
        for (d, m, q, x, _) in mats:
            O.linear(d, m, q, x)
    dt = time.perf_counter() - t0
    return dt, sum(b for *_, b in mats) * repeats


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    mats = oracle_layer_sample(which=("q",))
    for _ in range(args.warmup):
        time_oracle(mats)
    t, nbytes = 0.0, 0
    for _ in range(args.steps):
        dt, nb = time_oracle(mats)
        t += dt; nbytes += nb
    val = nbytes / t / 1e9
    sample = "per step: oracle dequant + fp64 mat-vec of one 4096x4096 2-bit matrix of the stack (M=1)"
    line = {"impl": "reference", "metric": "decode_weight_stream", "value": val, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_micro(args):
    """One kernel, small case, a few launches: what the ncu captures under profiles/ run."""
    import torch
    from paper_2605_24011_b200 import aq, synth, workloads
    torch.cuda.set_device(0)
    out = {"micro": args.micro, "bits": args.bits, "steps": args.steps, "warmup": args.warmup}
    if args.micro in ("pack", "pack_opt"):
        # set-up kernels: float32 weights (and Fisher scores) in, packed fragments out; HBM-bound on the 4 (8) B/weight read
        N, K = args.N or 16384, args.K or 8192
        Ws = [synth.weights_device(N, K, 7 + c) for c in range(2)]
        Fs = [(w * w * 2500.0 + 1e-4) for w in Ws] if args.micro == "pack_opt" else None
        held = []

        def fn(i):
            if len(held) >= 2:
                held.pop(0).free()
            if args.micro == "pack":
                held.append(aq.aq_pack(args.bits, 32, Ws[i % 2]))
            else:
                held.append(aq.aq_pack_opt(args.bits, 32, Ws[i % 2], Fs[i % 2], rounds=4))

        work, unit = N * K * (4.0 if args.micro == "pack" else 8.0) + N * K * (args.bits + 1) / 8, "GB/s"
        out.update({"N": N, "K": K, "note": "time includes handle allocation (cudaMalloc / cudaFree) on the host side"})
    elif args.micro in ("rbf_gram", "hsic"):
        # inter-tensor stage: kernel matrix of K calibration samples with d features (tensor-bound), HSIC over two such
        # matrices (HBM-bound: each read once)
        K, d = args.M or 4096, args.K or 11008
        if args.micro == "rbf_gram":
            As = [workloads.activations_device(K, d, torch.bfloat16, 11, c) for c in range(2)]
            G = torch.empty((K, K), dtype=torch.float32, device="cuda")
            fn = lambda i: aq.aq_rbf_gram(As[i % 2], float(d) ** 0.5, G=G)
            # inner products needed for a symmetric matrix: K (K + 1) / 2, each 2 d flops
            work, unit = float(K) * (K + 1) * d, "TFLOP/s"
        else:
            n_copies = max(2, int(300e6 // (K * K * 4)) + 1)
            A = workloads.activations_device(K, 512, torch.bfloat16, 12, 0)
            Gs = [aq.aq_rbf_gram(A, 512.0 ** 0.5) for _ in range(2 * n_copies)]
            res = torch.empty(1, dtype=torch.float64, device="cuda")
            fn = lambda i: aq.aq_hsic(Gs[2 * (i % n_copies)], Gs[2 * (i % n_copies) + 1], out=res)
            work, unit = 2.0 * K * K * 4, "GB/s"
        out.update({"K_samples": K, "d": d})
    elif args.micro == "decode_token":
        # one decoded token of the 7B-class stack with its attention (--K cached positions per block)
        prog0, out_buf0, names0, _, info0 = workloads.llama7b_decode_stack(n_layers=args.layers, seed=0)
        leg = decode_attn_leg(aq, info0, _peaks(), torch, context=args.K or 4096, steps=args.steps)
        out.update({"layers": args.layers, **leg})
        print(json.dumps(out))
        return
    elif args.micro == "attn_decode":
        # one decoded token of a 7B-class block (32 heads of 128) against --K cached positions; HBM-bound on the cache:
        # 2 (keys, values) x heads x positions x 128 x 2 bytes per call; caches rotate so that L2 does not hold them
        H, L = 32, args.K or 4096
        Hkv = args.N or 32                      # (--N: key/value heads, for grouped queries)
        per = 2 * Hkv * L * 128 * 2
        n_copies = max(1, int(600e6 // per))
        g = torch.Generator(device="cuda")
        g.manual_seed(11)
        caches = [(torch.randn((Hkv, L, 128), generator=g, device="cuda", dtype=torch.float16),
                   torch.randn((Hkv, L, 128), generator=g, device="cuda", dtype=torch.float16)) for _ in range(n_copies)]
        q = torch.randn((H, 128), generator=g, device="cuda", dtype=torch.float16)
        y = torch.empty((H, 128), dtype=torch.float16, device="cuda")
        scratch = torch.empty(aq.aq_attn_scratch_bytes(Hkv), dtype=torch.uint8, device="cuda")
        fn = lambda i: aq.aq_attn_decode(q, caches[i % n_copies][0], caches[i % n_copies][1], L, y, scratch)
        work, unit = per, "GB/s"
        out.update({"heads": H, "kv_heads": Hkv, "L": L, "copies": n_copies})
    elif args.micro in ("decode_linear", "prefill_linear", "dequant"):
        decode = args.micro == "decode_linear"
        M = args.M or (1 if decode else 512)
        N = args.N or (65536 if decode else 11008)
        K = args.K or (8192 if decode else 4096)
        dt = torch.float16 if decode else torch.bfloat16
        n_copies = 1 if decode else max(1, int(400e6 // (N * K * (args.bits + 1) // 8)))   # rotate past L2
        W = synth.weights_device(N, K, 7)
        hs = [aq.aq_pack(args.bits, 32, W) for _ in range(n_copies)]
        del W
        x = workloads.activations_device(M, K, dt, 9, M)
        if args.micro == "dequant":
            y = torch.empty((N, K), dtype=torch.float16, device="cuda")
            fn = lambda i: aq.aq_dequant(hs[i % n_copies], y)
            work, unit = N * K * (args.bits + 1) / 8 + 2.0 * N * K, "GB/s"
        else:
            y = torch.empty((M, N), dtype=torch.float32, device="cuda")
            fn = lambda i: aq.aq_linear(hs[i % n_copies], x, y)
            work, unit = (N * K * (args.bits + 1) / 8, "GB/s") if decode else (2.0 * M * N * K, "TFLOP/s")
        out.update({"M": M, "N": N, "K": K, "copies": n_copies})
        args.warmup = max(args.warmup, n_copies)   # every copy's handle has sized its scratch before the clock starts
    else:
        decode = args.micro == "decode_stack"
        M = args.M or (1 if decode else 512)
        prog, out_buf, names, _, info = workloads.llama7b_decode_stack(n_layers=args.layers, seed=0)
        ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
        dt = torch.float16 if decode else torch.bfloat16
        x0 = workloads.activations_device(M, 4096, dt, 3, 0)
        y = torch.empty((M, 4096), dtype=dt, device="cuda")
        fn = lambda i: aq.aq_stack_forward(prog, x0, y, out_buf, M, ws)
        work, unit = (info["packed_bytes"], "GB/s") if decode else (2.0 * M * info["weights"], "TFLOP/s")
        out.update({"M": M, "layers": args.layers})
    for i in range(args.warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        fn(args.warmup + i)
    e1.record()
    torch.cuda.synchronize()
    aq.aq_check()
    ms = e0.elapsed_time(e1) / args.steps
    out.update({"us_per_call": 1e3 * ms, "value": work / (ms * 1e-3) / (1e9 if unit == "GB/s" else 1e12), "unit": unit})
    if args.micro == "attn_decode":
        # the same calls recorded once into a CUDA graph and replayed: device time without the host's per-call cost
        n = max(16, min(args.steps, 64))
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for i in range(n):
                    fn(i)
        torch.cuda.synchronize()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(10):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        aq.aq_check()
        msg = e0.elapsed_time(e1) / (10 * n)
        out.update({"us_per_call_graph": 1e3 * msg, "value_graph": work / (msg * 1e-3) / 1e9})
    print(json.dumps(out))


def run_configs(args):
    """The five workload configurations, one timing each (CUDA events, cold weights where a case fits in L2)."""
    import torch
    torch.cuda.set_device(0)
    print(json.dumps(configs_leg(_peaks(), torch, None, None, None)))


def configs_leg(peaks, torch, prog7, out_buf7, info7):
    """One timing per workload configuration other than the headline one, each with its roofline fraction (HBM bytes
    for the decode-shaped ones, flops for the prefill-shaped ones).  prog7: the 7B-class stack when the caller has
    built it already (else it is built here)."""
    from paper_2605_24011_b200 import aq, programs, synth, workloads
    out = {"peaks": peaks}
    hbm, tf_peak = peaks["hbm_gbs"], peaks["bf16_tflops"]

    def timed_us(fn, steps, warm=3):
        return 1e3 * _timed(fn, steps, warm, torch) / steps

    # 1: single linear 4096 x 4096, 4-bit, x fp16 [1][4096]: dequant + linear M = 1, cold (rotating copies) and L2-hot
    W = synth.weights_device(4096, 4096, 0)
    hs = [aq.aq_pack(4, 32, W) for _ in range(24)]
    del W
    x = workloads.activations_device(1, 4096, torch.float16, 1, 0)
    y = torch.empty((1, 4096), dtype=torch.float16, device="cuda")
    wf = [torch.empty((4096, 4096), dtype=torch.float16, device="cuda") for _ in range(8)]
    i = [0]

    def lin_cold():
        aq.aq_linear(hs[i[0] % 24], x, y); i[0] += 1

    def deq_cold():
        aq.aq_dequant(hs[i[0] % 24], wf[i[0] % 8]); i[0] += 1

    pb = 4096 * 4096 * 5 // 8
    t_lc, t_lh = timed_us(lin_cold, 48), timed_us(lambda: aq.aq_linear(hs[0], x, y), 48)
    t_dc, t_dh = timed_us(deq_cold, 48), timed_us(lambda: aq.aq_dequant(hs[0], wf[0]), 48)

    # the same 48 cold calls recorded once into a CUDA graph and replayed: device time per call without the host's
    # per-call cost (a Python call through ctypes takes longer than this kernel)
    def graph_us(fn, calls):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            for _ in range(calls):
                fn()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(calls):
                    fn()
        torch.cuda.synchronize()
        return timed_us(graph.replay, 10) / calls

    i[0] = 0
    t_lg = graph_us(lin_cold, 48)
    i[0] = 0
    t_dg = graph_us(deq_cold, 48)
    out["config1"] = {"roofline": {"bound": "hbm", "achieved": pb / t_lg / 1e3, "peak": hbm, "unit": "GB/s", "frac": pb / t_lg / 1e3 / hbm,
                                   "what": "aq_linear M=1, 4096x4096 4-bit, cold L2 (24 packed copies in rotation), 48 calls "
                                           "replayed from a CUDA graph"},
                      "dequant_roofline": {"bound": "hbm", "achieved": (pb + 2 * 4096 * 4096) / t_dg / 1e3, "peak": hbm, "unit": "GB/s",
                                           "frac": (pb + 2 * 4096 * 4096) / t_dg / 1e3 / hbm,
                                           "what": "aq_dequant of the same matrix, 48 calls replayed from a CUDA graph"},
                      "linear_M1_us_graph": t_lg, "linear_M1_gbs_graph": pb / t_lg / 1e3, "dequant_us_graph": t_dg,
                      "dequant_gbs_graph": (pb + 2 * 4096 * 4096) / t_dg / 1e3,
                      "linear_M1_us_cold": t_lc, "linear_M1_gbs_cold": pb / t_lc / 1e3, "linear_M1_us_l2hot": t_lh,
                      "linear_M1_gbs_l2hot": pb / t_lh / 1e3, "dequant_us_cold": t_dc,
                      "dequant_gbs_cold": (pb + 2 * 4096 * 4096) / t_dc / 1e3, "dequant_us_l2hot": t_dh,
                      "note": "one aq_linear call = one launch (a CTA per 16-row tile writes its outputs itself); the "
                              "*_cold / *_l2hot times are eager calls from Python and include the host's per-call cost"}
    for h in hs:
        h.free()
    del wf

    # 2: LLaMA-2-7B MLP at 3-bit, M = 1 and M = 8 (weights 67.6 MB: L2-resident when repeated; 6 copies rotate)
    H, I = 4096, 11008
    sets = []
    for c in range(6):
        g = aq.aq_pack(3, 32, synth.weights_device(I, H, 20 + c))
        u = aq.aq_pack(3, 32, synth.weights_device(I, H, 30 + c))
        d = aq.aq_pack(3, 32, synth.weights_device(H, I, 40 + c))
        sets.append(programs.mlp_program(g, u, d, H, I) + ((g, u, d),))
    cfg2 = {}
    for M in (1, 8):
        ws = torch.empty(sets[0][0].workspace_bytes(M), dtype=torch.uint8, device="cuda")
        x0 = workloads.activations_device(M, H, torch.float16, 2, M)
        yo = torch.empty((M, H), dtype=torch.float16, device="cuda")

        def mlp():
            prog, ob = sets[i[0] % 6][0], sets[i[0] % 6][1]
            aq.aq_stack_forward(prog, x0, yo, ob, M, ws); i[0] += 1

        t = timed_us(mlp, 36, 12)
        i[0] = 0
        tg = graph_us(mlp, 36)   # (every set has run eagerly by now: the decode tables exist)
        cfg2[f"M{M}_us"] = t
        cfg2[f"M{M}_gbs"] = 3 * 22_544_384 / t / 1e3
        cfg2[f"M{M}_us_graph"] = tg
        cfg2[f"M{M}_roofline"] = {"bound": "hbm", "achieved": 3 * 22_544_384 / tg / 1e3, "peak": hbm, "unit": "GB/s",
                                  "frac": 3 * 22_544_384 / tg / 1e3 / hbm, "what": "36 passes replayed from a CUDA graph"}
    out["config2"] = cfg2
    for st in sets:
        for h in st[3]:
            h.free()
    del sets

    # 3 and 4: the 7B-class stack, M = 1 (fp16) and M = 512 (bf16); only M = 8 when the caller times those two itself
    if prog7 is None:
        prog, out_buf, names, _, info = workloads.llama7b_decode_stack(n_layers=32, seed=0)
        cases = ((1, torch.float16, "config3"), (8, torch.float16, "config3_M8"), (512, torch.bfloat16, "config4"))
    else:
        prog, out_buf, info = prog7, out_buf7, info7
        cases = ((8, torch.float16, "config3_M8"),)
    for M, dt, key in cases:
        ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
        x0 = workloads.activations_device(M, 4096, dt, 3, M, kind="vision_text" if M == 512 else "normal")
        yo = torch.empty((M, 4096), dtype=dt, device="cuda")
        t = timed_us(lambda: aq.aq_stack_forward(prog, x0, yo, out_buf, M, ws), 20 if M <= 8 else 5)
        out[key] = {"us_per_pass": t, "gbs": info["packed_bytes"] / t / 1e3, "tflops": 2.0 * M * info["weights"] / t / 1e6,
                    "mean_code_bits": info["mean_code_bits"]}
        if M <= 8:
            out[key]["roofline"] = {"bound": "hbm", "achieved": info["packed_bytes"] / t / 1e3, "peak": hbm, "unit": "GB/s",
                                    "frac": info["packed_bytes"] / t / 1e3 / hbm}
        else:
            out[key]["roofline"] = {"bound": "tensor", "achieved": 2.0 * M * info["weights"] / t / 1e6, "peak": tf_peak, "unit": "TFLOP/s",
                                    "frac": 2.0 * M * info["weights"] / t / 1e6 / tf_peak}
        del ws
    del prog

    # 5: Gemma-2B-shaped backbone, prefill M = 768 (bf16); action expert, 10 steps at M = 50
    prog, out_buf, names, _, info = workloads.gemma2b_stack(n_layers=18, seed=0)
    M = 768
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = workloads.activations_device(M, 2048, torch.bfloat16, 5, 0)
    yo = torch.empty((M, 2048), dtype=torch.bfloat16, device="cuda")
    t = timed_us(lambda: aq.aq_stack_forward(prog, x0, yo, out_buf, M, ws), 5)
    c5 = {"backbone_prefill_M768_us": t, "backbone_prefill_tflops": 2.0 * M * info["weights"] / t / 1e6,
          "backbone_mean_code_bits": info["mean_code_bits"],
          "backbone_roofline": {"bound": "tensor", "achieved": 2.0 * M * info["weights"] / t / 1e6, "peak": tf_peak, "unit": "TFLOP/s",
                                "frac": 2.0 * M * info["weights"] / t / 1e6 / tf_peak}}
    del prog, ws
    prog, out_buf, names, _, info = workloads.expert_stack(n_layers=18, seed=0)
    M = 50
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    xs = [workloads.activations_device(M, 1024, torch.bfloat16, 6, st) for st in range(10)]
    yo = torch.empty((M, 1024), dtype=torch.bfloat16, device="cuda")

    def ten_steps():
        for st in range(10):
            aq.aq_stack_forward(prog, xs[st], yo, out_buf, M, ws)

    t = timed_us(ten_steps, 5)
    c5.update({"expert_10_steps_M50_us": t, "expert_us_per_step": t / 10, "expert_gbs": 10 * info["packed_bytes"] / t / 1e3,
               "expert_tflops": 10 * 2.0 * M * info["weights"] / t / 1e6,
               "expert_note": "194.6 MB of packed weights per step: partly L2-resident across the 10 steps"})
    # the same ten steps recorded once into a CUDA graph (1440 launches) and replayed: what a control loop would do
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        ten_steps()
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            ten_steps()
    torch.cuda.synchronize()
    tg = timed_us(graph.replay, 5)
    c5["expert_roofline"] = {"bound": "hbm", "achieved": 10 * info["packed_bytes"] / t / 1e3, "peak": hbm, "unit": "GB/s",
                             "frac": 10 * info["packed_bytes"] / t / 1e3 / hbm,
                             "what": "bytes = packed weights per flow-matching step (M = 50: 2 M flops per weight is far below the "
                                     "tensor roofline, the step is bound by streaming the weights and by its 144 launches)"}
    c5.update({"expert_graph_10_steps_M50_us": tg, "expert_graph_us_per_step": tg / 10,
               "expert_graph_gbs": 10 * info["packed_bytes"] / tg / 1e3, "expert_graph_tflops": 10 * 2.0 * M * info["weights"] / tg / 1e6})
    out["config5"] = c5
    aq.aq_check()
    return out


WORKLOAD = ("7B-class decoder linear stack, M=1 decode: 32 layers x {q,k,v,o 4096x4096; gate,up 11008x4096; "
            "down 4096x11008}, per-matrix 2/3/4-bit (mean 2.5), blocks of 32 + fp16 scale/min, N(0,0.02) weights "
            "with 0.1% x20 outliers, x fp16 N(0,1)")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--layers", type=int, default=32, help="decoder layers (32 = the full workload)")
    ap.add_argument("--no-extras", action="store_true", help="skip prefill / dequant / oracle legs")
    ap.add_argument("--micro", choices=("decode_linear", "prefill_linear", "dequant", "decode_stack", "prefill_stack", "pack", "pack_opt", "rbf_gram", "hsic", "attn_decode", "decode_token"),
                    help="time one kernel on a small case (the command ncu captures are taken from) instead of the benchmark")
    ap.add_argument("--configs", action="store_true",
                    help="time all five workload configurations once each and print one JSON object (not the benchmark line)")
    ap.add_argument("--bits", type=int, default=2)
    ap.add_argument("--M", type=int, default=None)
    ap.add_argument("--N", type=int, default=None)
    ap.add_argument("--K", type=int, default=None)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.micro:
        run_micro(args)
        return
    if args.configs:
        run_configs(args)
        return

    import numpy as np
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2605_24011_b200 import aq, synth, workloads
    peaks = _peaks()
    warm = max(3, args.warmup)

    # ---- set-up (untimed): generate, pack, wire --------------------------------------------------
    prog, out_buf, names, _, info = workloads.llama7b_decode_stack(n_layers=args.layers, seed=0)
    M = 1
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = workloads.activations_device(M, 4096, torch.float16, 3, 0)
    out = torch.empty((M, 4096), dtype=torch.float16, device="cuda")
    x0_host = x0.cpu().pin_memory()
    out_host = torch.empty_like(out, device="cpu").pin_memory()
    packed = info["packed_bytes"]

    def step():
        aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)

    def step_e2e():
        x0.copy_(x0_host, non_blocking=True)
        aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
        out_host.copy_(out, non_blocking=True)

    # ---- timed: device-resident, then end to end ---------------------------------------------------
    sampler = ClockSampler(local)
    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler.start()
    l0 = aq.aq_kernel_launches()
    ms = _timed(step, args.steps, 0, torch)
    launches = aq.aq_kernel_launches() - l0
    if dist:
        dist.barrier()
    ms_e2e = _timed(step_e2e, args.steps, 3, torch)
    clocks = sampler.stop()
    aq.aq_check()
    # the same matrices wired without the chain (every linear reads the program input): the streaming upper bound of the
    # chained pass above; reported beside it, not as the headline
    from paper_2605_24011_b200 import programs
    prog_i, out_i, _ = programs.independent_program(info["layers"])
    ws_i = torch.empty(prog_i.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    y_i = torch.empty((M, prog_i.buf_width[out_i]), dtype=torch.float16, device="cuda")
    l1 = aq.aq_kernel_launches()
    n_i = max(10, args.steps // 5)
    ms_i = _timed(lambda: aq.aq_stack_forward(prog_i, x0, y_i, out_i, M, ws_i), n_i, 3, torch)
    launches_i = (aq.aq_kernel_launches() - l1) / (n_i + 3)
    aq.aq_check()
    del ws_i, y_i
    ms, ms_e2e = reduce_max([ms, ms_e2e], dist, "cuda")
    ms_step = ms / args.steps
    value = whole_job_gbs(world, packed, ms_step)
    e2e = whole_job_gbs(world, packed, ms_e2e / args.steps)

    line = {
        "metric": "decode_weight_stream", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": args.layers, "M": 1, "packed_bytes_per_step": packed,
                   "mean_code_bits": info["mean_code_bits"], "stored_bits_per_weight": 8.0 * packed / info["weights"],
                   "l2": "inputs larger than L2: every step streams all packed weights (>> 126 MB) once",
                   "parallelism": "replicas only (one GPU per replica, no collective)"},
        "clocks": clocks,
        "e2e": {"value": e2e, "unit": "GB/s", "h2d_bytes_per_step": int(x0_host.numel() * 2),
                "d2h_bytes_per_step": int(out_host.numel() * 2), "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "us_per_decode_pass": 1e3 * ms_step,
        "independent_inputs": {"value": packed / (ms_i / n_i * 1e-3) / 1e9, "unit": "GB/s", "us_per_pass": 1e3 * ms_i / n_i,
                               "frac_of_hbm_peak": packed / (ms_i / n_i * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "launches_per_pass": launches_i,
                               "note": "same matrices, every linear reads the program input (no dependency chain): rank 0's own timing"},
        "pct_of_nominal_hbm": 100.0 * (value / world) / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "achieved": value / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": (value / world) / peaks["hbm_gbs"], "traffic": DECODE_TRAFFIC_BYTES,
                     "peak_source": peaks["source"],
                     "kernel": "decode_stack_kernel (one launch per pass; time = whole pass incl. its two glue kernels)",
                     "traffic_note": "dram bytes of the 4-layer ncu capture scaled by packed bytes to 32 layers",
                     "algorithmic_bytes_per_step": packed},
    }

    if world == 1 and rank == 0 and not args.no_extras:
        line["prefill"] = prefill_leg(aq, workloads, prog, out_buf, info, peaks, torch, local)
        line["dequant"] = dequant_leg(aq, synth, peaks, torch)
        line["attn_decode"] = attn_leg(aq, peaks, torch)
        if args.layers == 32:
            line["decode_with_attention"] = decode_attn_leg(aq, info, peaks, torch)
        if args.layers == 32:
            line["configs"] = configs_leg(peaks, torch, prog, out_buf, info)
        cores = len(os.sched_getaffinity(0))
        mats = oracle_layer_sample()
        dt, nb = time_oracle(mats, repeats=7)
        line["cpu_baseline"] = {"value": nb / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "seconds": dt,
                                "sample": "7 passes over one 7B-shaped layer (7 matrices, 202M weights, M=1): "
                                          "oracle dequant + fp64 mat-vec"}
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of the decode kernel per stack pass, from the ncu capture summarised in
# profiles/decode_stack_kernel_7b_4layers_M1.md: 355,754,752 + 3,822,848 bytes for the first 4 layers (354,172,928
# packed bytes), times 8 for the 32 layers (every byte is read once, so traffic grows with the packed bytes).
# Set to None whenever the kernel changes, until the capture has been taken again.
DECODE_TRAFFIC_BYTES = 8 * (355_754_752 + 3_822_848)
# gemm_kernel (profiles/gemm_kernel_11008x4096_M512_2bit.md): 21,212,160 + 19,456 bytes of DRAM traffic for one 11008 x 4096
# 2-bit launch (16,908,288 packed bytes), scaled by packed bytes to the 224 matrices of one pass
PREFILL_TRAFFIC_BYTES = round(2_833_383_424 * (21_212_160 + 19_456) / 16_908_288)


def prefill_leg(aq, workloads, prog, out_buf, info, peaks, torch, gpu_index=0):
    """Same stack, M = 512 prefill: 256 vision-like rows + 256 text rows, bf16.  The leg is a burst (a quarter of a
    second), so its roofline fraction divides by the measured burst peak; the fraction of the sustained peak (what a
    seconds-long GEMM loop holds under the power cap) is given beside it."""
    M = 512
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = workloads.activations_device(M, 4096, torch.bfloat16, 4, 0, kind="vision_text")
    out = torch.empty((M, 4096), dtype=torch.bfloat16, device="cuda")

    def step():
        aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)

    n_pass = 25
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_index)
    sampler.start()
    l0 = aq.aq_kernel_launches()
    ms = _timed(step, n_pass, 0, torch) / n_pass
    launches = (aq.aq_kernel_launches() - l0) // n_pass
    clocks = sampler.stop()
    aq.aq_check()
    flops = 2.0 * M * info["weights"]
    tf = flops / (ms * 1e-3) / 1e12
    return {"workload": "same stack, M=512 (256 vision rows N(0,1)*U(0.5,2) + 256 text rows), bf16, dequant->tcgen05 GEMM",
            "ms_per_pass": ms, "tflops": tf, "pct_of_nominal_bf16": 100.0 * tf / NOMINAL_BF16_TFLOPS,
            "gpu_launches_per_pass": int(launches), "passes_timed": n_pass, "clocks": clocks,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"],
                         "frac_of_sustained_peak": tf / (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]),
                         "traffic": PREFILL_TRAFFIC_BYTES, "traffic_note": "dram bytes of the one-launch ncu capture (11008 x 4096) scaled by packed bytes to the pass",
                         "peak_source": peaks["source"] + " (burst peak: the leg lasts about 0.2 s)",
                         "kernel": "gemm_kernel (128 grouped launches per pass; time = whole pass incl. staging kernels)"}}


def attn_leg(aq, peaks, torch):
    """One decoded token's attention over a key/value cache (32 heads of 128, fp16) at 4096 and 16384 positions: HBM-bound
    on the cache bytes; the calls are replayed from a CUDA graph (device time), caches rotate past L2."""
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    H = 32
    q = torch.randn((H, 128), generator=g, device="cuda", dtype=torch.float16)
    y = torch.empty((H, 128), dtype=torch.float16, device="cuda")
    scratch = torch.empty(aq.aq_attn_scratch_bytes(H), dtype=torch.uint8, device="cuda")
    out = {"workload": "aq_attn_decode, 32 heads of 128, fp16, one token against L cached positions, caches cold (in rotation)"}
    for L in (4096, 16384):
        per = 2 * H * L * 128 * 2
        n = max(2, int(600e6 // per))
        caches = [(torch.randn((H, L, 128), generator=g, device="cuda", dtype=torch.float16),
                   torch.randn((H, L, 128), generator=g, device="cuda", dtype=torch.float16)) for _ in range(n)]
        calls = 4 * n
        fn = lambda i: aq.aq_attn_decode(q, caches[i % n][0], caches[i % n][1], L, y, scratch)
        for i in range(n):
            fn(i)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for i in range(calls):
                    fn(i)
        torch.cuda.synchronize()
        us = 1e3 * _timed(graph.replay, 10, 3, torch) / (10 * calls)
        aq.aq_check()
        gbs = per / us / 1e3
        out[f"L{L}"] = {"us_per_call": us, "gbs": gbs,
                        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                     "traffic": 67_175_680 + 434_688 if L == 4096 else None, "peak_source": peaks["source"],
                                     "kernel": "attn_decode_kernel"}}
        del caches
    return out


def decode_attn_leg(aq, info, peaks, torch, context=4096, steps=30):
    """One decoded token of the same 7B-class stack WITH its attention: per block q, k, v -> rotation, cache append,
    attention over `context` cached positions -> W_o ... (aq_stack_forward_attn: one launch of the decode kernel per
    stretch of linears between two attention steps).  Bytes = packed weights + the keys and values read."""
    from paper_2605_24011_b200 import programs, workloads
    H = 32
    prog, out_buf, names, attn = programs.block_program_attn(info["layers"], H, H)
    g = torch.Generator(device="cuda")
    g.manual_seed(13)
    Lmax = context + 8
    for t in attn:
        t["k_cache"] = torch.randn((H, Lmax, 128), generator=g, device="cuda", dtype=torch.float16)
        t["v_cache"] = torch.randn((H, Lmax, 128), generator=g, device="cuda", dtype=torch.float16)
    ws = torch.empty(prog.workspace_bytes(1), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(aq.aq_stack_attn_scratch_bytes(H, H, 1), dtype=torch.uint8, device="cuda")
    x0 = workloads.activations_device(1, 4096, torch.float16, 3, 1)
    y = torch.empty((1, 4096), dtype=torch.float16, device="cuda")
    pos = context - 1
    fn = lambda: aq.aq_stack_forward_attn(prog, attn, pos, x0, y, out_buf, 1, ws, scratch)
    l0 = aq.aq_kernel_launches()
    fn()
    launches = aq.aq_kernel_launches() - l0
    ms = _timed(fn, steps, 3, torch) / steps
    aq.aq_check()
    # the same token replayed from a CUDA graph: device time without the host's share of 98 launches
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            fn()
    torch.cuda.synchronize()
    ms_graph = _timed(graph.replay, steps, 3, torch) / steps
    aq.aq_check()
    kv = len(attn) * 2 * H * context * 128 * 2
    byts = info["packed_bytes"] + kv
    for t in attn:
        del t["k_cache"], t["v_cache"]
    return {"workload": f"the same stack with attention over {context} cached positions per block (32 heads of 128, fp16 caches), M = 1",
            "us_per_token": 1e3 * ms, "gbs": byts / ms / 1e6, "us_per_token_graph": 1e3 * ms_graph, "gbs_graph": byts / ms_graph / 1e6,
            "kv_bytes": kv, "launches_per_token": launches,
            "roofline": {"bound": "hbm", "achieved": byts / ms_graph / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": byts / ms_graph / 1e6 / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                         "what": "graph replay",
                         "kernel": "decode_stack_kernel (33 launches) + attn_decode_kernel (32) + attn_prepare_kernel (32)"}}


def dequant_leg(aq, synth, peaks, torch):
    """Standalone dequant, cold L2 (packed copies and outputs in rotation): the single 4096 x 4096 4-bit linear of the
    small configuration (launch-latency sized: 44 MB per call) and a 16384 x 8192 matrix that amortises the launch."""
    def run(N, K, n_packed, n_out, steps):
        W = synth.weights_device(N, K, 1)
        hs = [aq.aq_pack(4, 32, W) for _ in range(n_packed)]
        del W
        outs = [torch.empty((N, K), dtype=torch.float16, device="cuda") for _ in range(n_out)]
        i = [0]

        def step():
            aq.aq_dequant(hs[i[0] % n_packed], outs[i[0] % n_out])
            i[0] += 1

        ms = _timed(step, steps, 8, torch) / steps
        for h in hs:
            h.free()
        nbytes = N * K * 5 // 8 + N * K * 2
        return ms, nbytes / (ms * 1e-3) / 1e9

    ms_s, gbs_s = run(4096, 4096, 24, 8, 48)
    ms_l, gbs_l = run(16384, 8192, 3, 2, 12)
    return {"workload": "aq_dequant 4-bit -> fp16, cold L2: 16384x8192 (roofline) and 4096x4096 (the single-linear configuration)",
            "us_per_call": 1e3 * ms_l, "gbs": gbs_l, "us_per_call_4096": 1e3 * ms_s, "gbs_4096": gbs_s,
            "roofline": {"bound": "hbm", "achieved": gbs_l, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs_l / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                         "kernel": "dequant_kernel, 16384x8192"}}


if __name__ == "__main__":
    main()
