#!/usr/bin/env python
"""Benchmark of the decomposed-layer training step on B200.

Default workload: the BERT-base-shaped block (four 768->768 layers at r=192, 768->3072 and
3072->768 at r=384, M = 4096 tokens, bf16 with fp32 accumulation), forward + backward of every
layer per step, sequential freezing alternating U-frozen / V-frozen every step.

One JSON line on stdout (rank 0).  `value` is tokens/s with inputs resident in HBM; `e2e` is the
same step with the activations copied from pinned host memory and the weight gradients copied
back inside the timed region; `roofline` is the dominant kernel, timed alone with CUDA events;
`cpu_baseline` is the fp64 CPU oracle timed on this machine's host cores.

--config picks the workload: c1 (the default, above); c0 the single fp32 layer (256 x 512 -> 512, r = 40, three
masks); c2 the rank-quantization sweep on the 4096 x 4096 layer at 8192 tokens (every rank packed and rounded up to
8 / 64 / 128, no freezing and V frozen, beside the dense layer); c3 the ResNet-50-stage-3-shaped Tucker-2
convolution; c4 the decomposed layers of a 12-block GPT-2-medium-shaped stack beside the undecomposed stack.
Each prints the same kind of line for its own headline variant, with every variant it timed under "variants".
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes of one launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of an ncu capture of
# the 768->3072, r=384 forward; summary in profiles/chain_kernel_ffn1_forward.md).  It is reported only while the
# kernel's sources still have the digest the capture was taken with.
NCU_TRAFFIC = {"digest": "43a48a7824f353d6", "bytes_per_launch": 9320192, "l2_to_sm_bytes_per_launch": 129171456,
               "note": "DRAM reads of the launch (X and the weights once); its 25 MB of output were still in the 126 MB L2 when "
                       "the counters stopped, so this is below the algorithmic bytes and says only that nothing is re-read from HBM"}
KERNEL_SOURCES = ("paper_2309_03824_b200/csrc/chain.cu", "paper_2309_03824_b200/csrc/ptx.cuh")


def kernel_digest():
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(hashlib.sha256(f.read()).digest())
    return h.hexdigest()[:16]
L2_BYTES = 126 * 1024 * 1024


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ---- algorithmic work of one layer (what the method must do; every tensor once) ------------------
def layer_flops(M, K, N, r, freeze, which):
    fwd = 2 * M * r * (K + N)
    bwd = 2 * M * N * r + 2 * M * r * K + (0 if freeze == 1 else 2 * M * N * r) + (0 if freeze == 2 else 2 * M * K * r)
    return {"fwd": fwd, "bwd": bwd, "both": fwd + bwd}[which]


def layer_bytes(M, K, N, r, freeze, which, e=2):
    fwd = e * (M * K + K * r + N * r + N + M * N + (0 if freeze == 1 else M * r))
    bwd = e * (M * N + N * r + K * r + M * K)
    if freeze != 1:
        bwd += e * (M * r + N * r + N)
    if freeze != 2:
        bwd += e * (M * K + K * r)
    return {"fwd": fwd, "bwd": bwd, "both": fwd + bwd}[which]


# ---- clocks -----------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, t0, t1):
        sm, mx, reasons = [], 0, set()
        for ts, line in self.rows:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                clk, cmax = float(f[1]), float(f[2])
            except ValueError:
                continue
            mx = max(mx, cmax)
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(clk)
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        if not sm:      # timed region shorter than the sampling period: take every sample there is
            for ts, line in self.rows:
                f = [x.strip() for x in line.split(",")]
                try:
                    sm.append(float(f[1]))
                except Exception:
                    pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(ms, world, device):
    """A timing in ms -> the slowest rank's (all-reduce MAX over the process group); identity for one rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank, world, ms_per_step):
    """Weak scaling: every rank runs the same workload; throughput counts all ranks' tokens over the slowest rank's time."""
    return tokens_per_rank * world / (ms_per_step * 1e-3)


# ---- the oracle, timed (CPU baseline / reference arm) ------------------------------------------------
def oracle_block_seconds(layers_np, min_seconds, max_reps=400):
    """Forward + backward of the whole block in the fp64 oracle, alternating masks; returns
    (seconds per step, steps run, threads used)."""
    from oracle import lrd_oracle as o
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    t0 = time.perf_counter()
    reps = 0
    while True:
        freeze = o.FREEZE_U if reps % 2 == 0 else o.FREEZE_V
        for c in layers_np:
            Z, _ = o.linear_fwd(c["X"], c["V"], c["U"], c["b"])
            o.linear_bwd(c["dY"], c["X"], c["V"], c["U"], Z, freeze)
        reps += 1
        if (time.perf_counter() - t0 >= min_seconds and reps % 2 == 0) or reps >= max_reps:
            break
    return (time.perf_counter() - t0) / reps, reps, threads


def make_layers_numpy(factorize):
    from paper_2309_03824_b200 import workloads as wl
    cases = []
    for i, (name, K, N, r) in enumerate(wl.C1_BERT_LAYERS):
        c = wl.linear_case(wl.C1_M, K, N, r, "bf16", 1000 + 10 * i, wl.W_STD_TRANSFORMER, factorize)
        c["name"] = name
        cases.append(c)
    return cases


def config_dict(extra=None):
    from paper_2309_03824_b200 import workloads as wl
    cfg = {"workload": "configs[1]: BERT-base-shaped decomposed block, 4x(768->768,r=192)+(768->3072,r=384)+(3072->768,r=384), "
                       "M=4096 tokens, fwd+bwd, sequential freezing alternating U-frozen/V-frozen per step",
           "tokens_per_step": wl.C1_M, "layers": len(wl.C1_BERT_LAYERS), "ranks_quantized_to": 64}
    if extra:
        cfg.update(extra)
    return cfg


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2309_03824_b200 import workloads as wl

    def np_factors(W, r):      # input construction only (the oracle's own SVD is pinned by its tests)
        Uf, s, Vt = np.linalg.svd(W, full_matrices=False)
        root = np.sqrt(s[:r])
        return Vt[:r].T * root, Uf[:, :r] * root

    cases = make_layers_numpy(np_factors)
    for c in cases:
        for k in ("X", "V", "U", "b", "dY"):
            c[k] = c[k].astype(np.float64)
    for _ in range(max(args.warmup, 0)):
        oracle_block_seconds(cases, 0.0, max_reps=2)
    steps = max(args.steps, 2)
    steps += steps % 2
    t0 = time.perf_counter()
    sec, reps, threads = oracle_block_seconds(cases, 1e9, max_reps=steps)
    total = time.perf_counter() - t0
    val = wl.C1_M / sec
    line = {"impl": "reference", "metric": "LRD layer fwd+bwd tokens/s", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": reps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict({"sample": "full block, M=4096, every layer, both masks alternating"}),
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                             "sample": f"{reps} full steps of the block at M=4096 ({total:.1f} s)"},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)



# ---- pieces shared by the workloads other than the default one -------------------------------------------
def time_graph(torch, fn, sets, reps=10, rounds=1, repeats=5):
    """Seconds per call of fn(s), s cycling over `sets` buffer sets: a CUDA graph of rounds x sets calls replayed
    `reps` times per repeat, median over `repeats` repeats; also (min, max) over the repeats."""
    for s in range(sets):
        fn(s)
    torch.cuda.synchronize()
    side, g = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(rounds):          # a graph launch leaves the device idle for ~14 us: more rounds per graph for short steps
                for s in range(sets):
                    fn(s)
    torch.cuda.synchronize()
    g.replay()
    out = []
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) * 1e-3 / (reps * rounds * sets))
    out.sort()
    return out[len(out) // 2], (out[0], out[-1])


def time_e2e(torch, step, h2d, d2h, steps):
    """Seconds per step with the step's inputs copied from pinned host memory first and its results copied back after,
    every step, all inside the timed region (one stream, in order).  h2d / d2h: lists of (dst, src) tensor pairs."""
    def one():
        for dst, src in h2d:
            dst.copy_(src, non_blocking=True)
        step()
        for dst, src in d2h:
            dst.copy_(src, non_blocking=True)
    for _ in range(3):
        one()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    nbytes = lambda pairs: int(sum(d.numel() * d.element_size() for d, _ in pairs))
    return e0.elapsed_time(e1) * 1e-3 / steps, nbytes(h2d), nbytes(d2h)


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def time_oracle(fn, min_seconds, max_reps=100000):
    """Seconds per call of fn() (the oracle as it stands), run for at least min_seconds."""
    fn()
    t0 = time.perf_counter()
    reps = 0
    while True:
        fn()
        reps += 1
        if time.perf_counter() - t0 >= min_seconds or reps >= max_reps:
            break
    return (time.perf_counter() - t0) / reps, reps


def dense_flops_bytes(M, K, N, e=2):
    return 6 * M * K * N, e * (M * K + K * N + N + M * N) + e * (M * N + K * N + M * K) + e * (M * K + K * N + N)


def roof_of(flops, nbytes, sec, peaks):
    t_t, t_h = flops / (peaks["bf16_tflops"] * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)
    if t_t >= t_h:
        return {"bound": "tensor", "achieved": flops / sec / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": t_t / sec, "traffic": None}
    return {"bound": "hbm", "achieved": nbytes / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": t_h / sec, "traffic": None}


def tucker_flops_bytes(P, C, S, r1, r2, freeze, e=2):
    """Algorithmic work of one forward + backward of the Tucker-2 layer over P pixels (every tensor once)."""
    core = 2 * P * 9 * r1 * r2
    fwd = 2 * P * (C * r1 + r2 * S) + core
    bwd = fwd                                                     # data path
    if freeze != 2:                                               # core unfrozen: filter gradient
        bwd += core
    if freeze != 1:                                               # 1x1 factors unfrozen: dA, dB
        bwd += 2 * P * (C * r1 + r2 * S)
    w = C * r1 + 9 * r1 * r2 + S * r2
    by = e * (P * (C + S) + w + S) + e * (P * (S + C) + w)
    if freeze != 2:
        by += e * (2 * P * r1 + 9 * r1 * r2)                      # Z1 saved and read back, dG
    if freeze != 1:
        by += e * (2 * P * r2 + P * C + C * r1 + S * r2 + S)      # Z2 saved and read back, X read again, dA, dB, db
    return fwd + bwd, by


def emit(args, world, name, workload, tokens, sec, spread, dtype, roof, cpu, e2e, launches, clocks, peak_src, variants, extra=None):
    cfg = {"workload": workload, "tokens_per_step": tokens, "parallelism": f"replicas x{world}" if world > 1 else "single GPU"}
    if extra:
        cfg.update(extra)
    line = {"metric": "LRD layer fwd+bwd tokens/s", "value": tokens * world / sec, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic", "config": cfg,
            "repeats": {"n": 5, "min_ms": spread[0] * 1e3, "max_ms": spread[1] * 1e3, "reported": "median"},
            "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "peaks": peak_src,
            "variants": variants}
    print(json.dumps(line), flush=True)


def run_other(args):
    """Workloads c0, c2, c3, c4 (single rank's work; under torchrun every rank runs it and rank 0 reports)."""
    import torch
    import torch.distributed as dist
    from paper_2309_03824_b200 import build as lrd_build
    lrd_build.build()
    from paper_2309_03824_b200 import binding as b
    from paper_2309_03824_b200 import decompose
    from paper_2309_03824_b200 import workloads as wl
    from oracle import lrd_oracle as o

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU path exists)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peak_src = load_peaks()
    b.lrd_set_path({"auto": 0, "general": 1, "unfused": 2, "fused": 3}[args.path])
    bf = torch.bfloat16
    reps = max(2, args.steps // 4)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    t_begin = time.time()
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    threads = oracle_threads()
    MASK = {0: "none", 1: "U", 2: "V"}

    def linear_state(M, K, N, r, dtype, sets, packed_ld=True, gen=None, case=None):
        """Device tensors of one layer: seeded draws made on the device (timing), or a host-made case (oracle comparison)."""
        tdt = bf if dtype == "bf16" else torch.float32
        code = b.LRD_BF16 if dtype == "bf16" else b.LRD_F32
        L = {"M": M, "K": K, "N": N, "r": r, "desc": b.linear_desc(M, K, N, r, code), "tdt": tdt}
        if case is not None:
            L["V"], L["U"], L["b"] = (torch.from_numpy(case[k]).to("cuda", tdt) for k in ("V", "U", "b"))
            hX, hdY = torch.from_numpy(case["X"]).to(tdt).pin_memory(), torch.from_numpy(case["dY"]).to(tdt).pin_memory()
        else:
            rn = lambda *sh, std=1.0: (torch.randn(*sh, device="cuda", generator=gen) * std).to(tdt)
            L["V"], L["U"], L["b"] = rn(K, r, std=0.02), rn(N, r, std=0.02), rn(N, std=0.1)
            hX, hdY = rn(M, K).cpu().pin_memory(), rn(M, N).cpu().pin_memory()
        L["hX"], L["hdY"] = hX, hdY
        L["sets"] = [dict(X=hX.to("cuda"), dY=hdY.to("cuda"), Y=torch.empty(M, N, dtype=tdt, device="cuda"),
                          Z=torch.empty(M, r, dtype=tdt, device="cuda"), dX=torch.empty(M, K, dtype=tdt, device="cuda")) for _ in range(sets)]
        L["dU"], L["dV"], L["db"] = (torch.empty(*sh, dtype=tdt, device="cuda") for sh in ((N, r), (K, r), (N,)))
        L["hdU"], L["hdV"], L["hdb"] = (torch.empty(*sh, dtype=tdt).pin_memory() for sh in ((N, r), (K, r), (N,)))
        nws = max(b.lrd_linear_workspace_bytes(L["desc"], 0, 0), b.lrd_linear_workspace_bytes(L["desc"], 0, 1), 256)
        L["ws"] = torch.empty(nws, dtype=torch.uint8, device="cuda")
        return L

    def lin_step(L, s, f):
        st = L["sets"][s]
        b.lrd_linear_fwd(L["desc"], st["X"], L["V"], L["U"], L["b"], st["Y"], None if f == 1 else st["Z"], f, L["ws"])
        b.lrd_linear_bwd(L["desc"], st["dY"], None if f == 2 else st["X"], L["V"], L["U"], None if f == 1 else st["Z"], st["dX"],
                         None if f == 1 else L["dU"], None if f == 2 else L["dV"], None if f == 1 else L["db"], f, L["ws"])

    def lin_copies(L, f):
        st = L["sets"][0]
        h2d = [(st["X"], L["hX"]), (st["dY"], L["hdY"])]
        d2h = ([(L["hdU"], L["dU"]), (L["hdb"], L["db"])] if f != 1 else []) + ([(L["hdV"], L["dV"])] if f != 2 else [])
        return h2d, d2h

    def count(fn):
        n0 = b.lrd_launch_count()
        fn()
        return b.lrd_launch_count() - n0

    variants = []

    def finish(name, workload, tokens, sec, spread, dtype, roof, cpu, e2e_t, launches, extra=None):
        if b.lrd_check_device_status() != b.LRD_OK:
            raise SystemExit("device-side wait timed out")
        for v in variants:
            log(json.dumps(v))
        ms = max_over_ranks(sec * 1e3, world, "cuda")
        if rank == 0:
            sampler.stop()
            clocks = sampler.summary(t_begin, time.time())
            e2e = {"value": tokens * world / e2e_t[0], "unit": "tokens/s", "h2d_bytes_per_step": e2e_t[1], "d2h_bytes_per_step": e2e_t[2]}
            emit(args, world, name, workload, tokens, ms * 1e-3, spread, dtype, roof, cpu, e2e, launches, clocks, peak_src, variants, extra)
        if world > 1:
            dist.destroy_process_group()

    # ------------------------------------------------------------------------------------------------ c0
    if args.config == "c0":
        c = wl.C0_LINEAR
        case = wl.linear_case(c["M"], c["K"], c["N"], c["r"], "f32", 0, c["w_std"], decompose.svd_factors, w_seed=0)
        S = 64                                                    # 64 sets x 2.6 MB > L2
        L = linear_state(c["M"], c["K"], c["N"], c["r"], "f32", S, case=case)
        secs = []
        for f in (0, 1, 2):
            sec, spread = time_graph(torch, lambda s, f=f: lin_step(L, s, f), S, reps=reps, rounds=1)
            fl, by = layer_flops(c["M"], c["K"], c["N"], c["r"], f, "both"), layer_bytes(c["M"], c["K"], c["N"], c["r"], f, "both", e=4)
            variants.append({"variant": f"freeze={MASK[f]}", "us": sec * 1e6, "tokens_per_s": c["M"] / sec, "gflops": fl / sec / 1e9,
                             "gbs": by / sec / 1e9, "kernels": count(lambda: lin_step(L, 0, f))})
            secs.append((sec, spread, by))
        sec = sum(x[0] for x in secs) / 3
        by = sum(x[2] for x in secs) / 3
        roof = {"bound": "hbm", "achieved": by / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": by / sec / 1e9 / peaks["hbm_gbs"],
                "traffic": None, "note": "fp32 FMA kernels, launch-latency bound at this size: time and GB/s are reported, there is no tensor-core fraction"}
        h2d, d2h = lin_copies(L, 0)
        e2e_t = time_e2e(torch, lambda: lin_step(L, 0, 0), h2d, d2h, max(10, args.steps))
        cpu = None
        if want_cpu:
            cc = {k: case[k].astype(np.float64) for k in ("X", "V", "U", "b", "dY")}

            def cpu_step():
                for f in (0, 1, 2):
                    Z, _ = o.linear_fwd(cc["X"], cc["V"], cc["U"], cc["b"])
                    o.linear_bwd(cc["dY"], cc["X"], cc["V"], cc["U"], Z, f)
            csec, creps = time_oracle(cpu_step, 5.0)
            cpu = {"value": c["M"] / (csec / 3), "unit": "tokens/s", "cores": threads, "kind": "oracle",
                   "sample": f"{creps} x (forward + backward under the three masks) at full size"}
        return finish("c0", "configs[0]: single low-rank linear layer, fp32, X[256x512], W[512x512] -> r=40, fwd+bwd, mean of the masks none / U / V",
                      c["M"], sec, (min(x[1][0] for x in secs), max(x[1][1] for x in secs)), "f32", roof, cpu, e2e_t,
                      sum(v["kernels"] for v in variants) * args.steps // 3, {"l2": f"cycling {S} buffer sets"})

    # ------------------------------------------------------------------------------------------------ c2
    if args.config == "c2":
        c = wl.C2_SWEEP
        M, K, N = c["M"], c["K"], c["N"]
        S = 2                                                     # 2 x 270 MB > L2
        gen = torch.Generator(device="cuda").manual_seed(2000)
        base = linear_state(M, K, N, 8, "bf16", S, gen=gen)       # activations shared by every rank of the sweep
        head = None
        todo, seen = [], set()
        for r0 in c["ranks"]:
            for label, mult in (("packed", 1), ("x8", 8), ("x64", 64), ("x128", 128)):
                r = r0 if mult == 1 else b.lrd_rank_quantize(r0, mult, b.LRD_ROUND_UP, K, N)
                if r not in seen:
                    seen.add(r)
                    todo.append((f"r={r0} {label}", r))
        for name, r in todo:
            L = dict(base)
            rn = lambda *sh, std=1.0: (torch.randn(*sh, device="cuda", generator=gen) * std).to(bf)
            L.update({"r": r, "desc": b.linear_desc(M, K, N, r, b.LRD_BF16), "V": rn(K, r, std=0.02), "U": rn(N, r, std=0.02)})
            L["sets"] = [dict(st, Z=torch.empty(M, r, dtype=bf, device="cuda")) for st in base["sets"]]
            L["dU"], L["dV"] = torch.empty(N, r, dtype=bf, device="cuda"), torch.empty(K, r, dtype=bf, device="cuda")
            nws = max(b.lrd_linear_workspace_bytes(L["desc"], 0, 0), b.lrd_linear_workspace_bytes(L["desc"], 0, 1), 256)
            L["ws"] = torch.empty(nws, dtype=torch.uint8, device="cuda")
            for f in (0, 2):
                sec, spread = time_graph(torch, lambda s, f=f: lin_step(L, s, f), S, reps=max(2, reps // 2))
                fl, by = layer_flops(M, K, N, r, f, "both"), layer_bytes(M, K, N, r, f, "both")
                rf = roof_of(fl, by, sec, peaks)
                v = {"variant": f"{name} freeze={MASK[f]}", "r": r, "us": sec * 1e6, "tokens_per_s": M / sec, "tflops": fl / sec / 1e12,
                     "bound": rf["bound"], "frac": rf["frac"], "kernels": count(lambda: lin_step(L, 0, f))}
                variants.append(v)
                if r == 256 and f == 0:
                    L["hdU"], L["hdV"] = torch.empty(N, r, dtype=bf).pin_memory(), torch.empty(K, r, dtype=bf).pin_memory()
                    head = (sec, spread, rf, v["kernels"], L)
        W = (torch.randn(N, K, device="cuda", generator=gen) * 0.02).to(bf)
        dW = torch.empty(N, K, dtype=bf, device="cuda")
        dd = b.linear_desc(M, K, N, 0, b.LRD_BF16)
        wsd = torch.empty(max(b.lrd_dense_workspace_bytes(dd, 1), 256), dtype=torch.uint8, device="cuda")

        def dense_step(s):
            st = base["sets"][s]
            b.lrd_dense_fwd(dd, st["X"], W, base["b"], st["Y"], wsd)
            b.lrd_dense_bwd(dd, st["dY"], st["X"], W, st["dX"], dW, base["db"], wsd)
        sec, spread = time_graph(torch, dense_step, S, reps=max(2, reps // 2))
        fl, by = dense_flops_bytes(M, K, N)
        rf = roof_of(fl, by, sec, peaks)
        variants.append({"variant": "dense 4096x4096", "r": 0, "us": sec * 1e6, "tokens_per_s": M / sec, "tflops": fl / sec / 1e12,
                         "bound": rf["bound"], "frac": rf["frac"], "kernels": count(lambda: dense_step(0))})
        sec, spread, roof, nk, L = head
        h2d, d2h = lin_copies(L, 0)
        e2e_t = time_e2e(torch, lambda: lin_step(L, 0, 0), h2d, d2h, max(4, args.steps // 4))
        cpu = None
        if want_cpu:
            Ms = 512
            cc = wl.random_factor_case(Ms, K, N, 256, "bf16", 2256)
            cc = {k: cc[k].astype(np.float64) for k in ("X", "V", "U", "b", "dY")}

            def cpu_step():
                Z, _ = o.linear_fwd(cc["X"], cc["V"], cc["U"], cc["b"])
                o.linear_bwd(cc["dY"], cc["X"], cc["V"], cc["U"], Z, 0)
            csec, creps = time_oracle(cpu_step, 8.0)
            cpu = {"value": Ms / csec, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                   "sample": f"scaled: {creps} x forward + backward of the r=256 layer on a slice of {Ms} of the {M} tokens (rows are independent)"}
        return finish("c2", "configs[2]: rank-quantization sweep, one 4096x4096 layer, M=8192 tokens, bf16; headline variant r=250 rounded up to 256 "
                      "(x8, x64 and x128 agree), fwd+bwd, nothing frozen; every rank, rounding and mask under 'variants'", M, sec, spread, "bf16", roof, cpu,
                      e2e_t, nk * args.steps, {"l2": f"cycling {S} activation buffer sets of 270 MB", "factors": "drawn directly on the device (timing only)"})

    # ------------------------------------------------------------------------------------------------ c3
    if args.config == "c3":
        c = wl.C3_TUCKER
        B, H, W_, C_, S_, r1, r2 = c["B"], c["H"], c["W"], c["C"], c["S"], c["r1"], c["r2"]
        P = B * H * W_
        case = wl.tucker_case(B, H, W_, C_, S_, r1, r2, c["k"], "bf16", 3000, decompose.tucker2_factors)
        NS = 12                                                   # 12 sets x 16 MB > L2
        desc = b.tucker2_desc(B, H, W_, C_, S_, r1, r2, b.LRD_BF16)
        dev = lambda a: torch.from_numpy(a).to("cuda", bf)
        A, G, Bm, bias = (dev(case[k]) for k in ("A", "G", "Bm", "b"))
        hX, hdY = torch.from_numpy(case["X"]).to(bf).pin_memory(), torch.from_numpy(case["dY"]).to(bf).pin_memory()
        sets = [dict(X=hX.to("cuda"), dY=hdY.to("cuda"), Y=torch.empty(B, H, W_, S_, dtype=bf, device="cuda"),
                     Z1=torch.empty(B, H, W_, r1, dtype=bf, device="cuda"), Z2=torch.empty(B, H, W_, r2, dtype=bf, device="cuda"),
                     dX=torch.empty(B, H, W_, C_, dtype=bf, device="cuda")) for _ in range(NS)]
        dA, dG, dB, db = (torch.empty(*sh, dtype=bf, device="cuda") for sh in ((C_, r1), (r2, 3, 3, r1), (S_, r2), (S_,)))
        hg = [torch.empty_like(t, device="cpu").pin_memory() for t in (dA, dG, dB, db)]
        ws = torch.empty(max(b.lrd_tucker2_workspace_bytes(desc, 0, 0), b.lrd_tucker2_workspace_bytes(desc, 0, 1), 256), dtype=torch.uint8, device="cuda")

        def tk_fwd(s, f):
            st = sets[s]
            b.lrd_tucker2_fwd(desc, st["X"], A, G, Bm, bias, st["Y"], None if f == 2 else st["Z1"], None if f == 1 else st["Z2"], f, ws)

        def tk_bwd(s, f):
            st = sets[s]
            b.lrd_tucker2_bwd(desc, st["dY"], None if f == 1 else st["X"], A, G, Bm, None if f == 2 else st["Z1"], None if f == 1 else st["Z2"],
                              st["dX"], None if f == 1 else dA, None if f == 2 else dG, None if f == 1 else dB, None if f == 1 else db, f, ws)

        def tk_step(s, f):
            tk_fwd(s, f)
            tk_bwd(s, f)
        TK = {0: "none", 1: "factors", 2: "core"}
        res = {}
        for f in (2, 1, 0):
            for what, fn in (("fwd", tk_fwd), ("bwd", tk_bwd), ("fwd+bwd", tk_step)):
                sec, spread = time_graph(torch, lambda s, f=f, fn=fn: fn(s, f), NS, reps=reps, rounds=2)
                res[(f, what)] = (sec, spread)
                variants.append({"variant": f"{what} frozen={TK[f]}", "us": sec * 1e6, "tokens_per_s": P / sec,
                                 "kernels": count(lambda: fn(0, f))})
        # headline: the workload's alternation, core frozen on even steps and the 1x1 factors on odd steps
        sec = 0.5 * (res[(2, "fwd+bwd")][0] + res[(1, "fwd+bwd")][0])
        spread = (min(res[(2, "fwd+bwd")][1][0], res[(1, "fwd+bwd")][1][0]), max(res[(2, "fwd+bwd")][1][1], res[(1, "fwd+bwd")][1][1]))
        fl = 0.5 * (tucker_flops_bytes(P, C_, S_, r1, r2, 2)[0] + tucker_flops_bytes(P, C_, S_, r1, r2, 1)[0])
        by = 0.5 * (tucker_flops_bytes(P, C_, S_, r1, r2, 2)[1] + tucker_flops_bytes(P, C_, S_, r1, r2, 1)[1])
        roof = roof_of(fl, by, sec, peaks)
        for v in variants:
            if v["variant"].startswith("fwd+bwd"):
                f = {"none": 0, "factors": 1, "core": 2}[v["variant"].split("=")[1]]
                w = tucker_flops_bytes(P, C_, S_, r1, r2, f)
                v["frac"] = roof_of(w[0], w[1], v["us"] * 1e-6, peaks)["frac"]
        st0 = sets[0]
        e2e_t = time_e2e(torch, lambda: (tk_step(0, 2), tk_step(0, 1)), [(st0["X"], hX), (st0["dY"], hdY)] * 2,
                         list(zip(hg, (dA, dG, dB, db))), max(4, args.steps // 2))
        e2e_t = (e2e_t[0] / 2, e2e_t[1] // 2, e2e_t[2] // 2)          # two steps (one per mask) per timed call
        cpu = None
        if want_cpu:
            Bs = 8
            cc = {k: case[k].astype(np.float64) for k in ("A", "G", "Bm", "b")}
            Xs, dYs = case["X"][:Bs].astype(np.float64), case["dY"][:Bs].astype(np.float64)

            def cpu_step():
                for f in (2, 1):
                    Z1, Z2, _ = o.tucker2_fwd(Xs, cc["A"], cc["G"], cc["Bm"], cc["b"])
                    o.tucker2_bwd(dYs, Xs, cc["A"], cc["G"], cc["Bm"], Z1, Z2, f)
            csec, creps = time_oracle(cpu_step, 8.0)
            cpu = {"value": Bs * H * W_ / (csec / 2), "unit": "tokens/s", "cores": threads, "kind": "oracle",
                   "sample": f"scaled: {creps} x (core-frozen step + factors-frozen step) on {Bs} of the {B} images (images are independent)"}
        nk = sum(v["kernels"] for v in variants if v["variant"] in ("fwd+bwd frozen=core", "fwd+bwd frozen=factors"))
        return finish("c3", "configs[3]: ResNet-50-stage-3-shaped Tucker-2 3x3 conv, bf16 NHWC, batch 64, 14x14, 256 -> r1=96 -> r2=96 -> 256, fwd+bwd, "
                      "core frozen on even steps / 1x1 factors frozen on odd steps; a token is a pixel", P, sec, spread, "bf16", roof, cpu, e2e_t,
                      nk * args.steps // 2, {"l2": f"cycling {NS} buffer sets of 16 MB"})

    # ------------------------------------------------------------------------------------------------ c4
    if args.config == "c4":
        M, NB = wl.C4_M, wl.C4_BLOCKS
        S = 2
        gen = torch.Generator(device="cuda").manual_seed(4000)
        acts = {name: linear_state(M, K, N, r, "bf16", S, gen=gen) for name, K, N, r in wl.C4_GPT_LAYERS}
        rn = lambda *sh, std=1.0: (torch.randn(*sh, device="cuda", generator=gen) * std).to(bf)
        blocks = []
        for _ in range(NB):                                       # every block has its own weights; activations are shared (timing)
            layers = []
            for name, K, N, r in wl.C4_GPT_LAYERS:
                L = dict(acts[name])
                L.update({"name": name, "V": rn(K, r, std=0.02), "U": rn(N, r, std=0.02), "W": rn(N, K, std=0.02),
                          "dW": acts[name].setdefault("dW", torch.empty(N, K, dtype=bf, device="cuda")),
                          "ddesc": b.linear_desc(M, K, N, 0, b.LRD_BF16)})
                L["wsd"] = acts[name].setdefault("wsd", torch.empty(max(b.lrd_dense_workspace_bytes(L["ddesc"], 1), 256), dtype=torch.uint8, device="cuda"))
                if not name.startswith(("attn_q", "attn_k", "attn_v")):
                    L["ws"] = torch.empty_like(acts[name]["ws"])
                layers.append(L)
            blocks.append(layers)

        def g_call(Ls, s, f, fwd):
            sts = [L["sets"][s] for L in Ls]
            if fwd:
                b.lrd_linear_group_fwd([L["desc"] for L in Ls], [x["X"] for x in sts], [L["V"] for L in Ls], [L["U"] for L in Ls],
                                       [L["b"] for L in Ls], [x["Y"] for x in sts], None if f == 1 else [x["Z"] for x in sts], f, [L["ws"] for L in Ls])
            else:
                b.lrd_linear_group_bwd([L["desc"] for L in Ls], [x["dY"] for x in sts], None if f == 2 else [x["X"] for x in sts],
                                       [L["V"] for L in Ls], [L["U"] for L in Ls], None if f == 1 else [x["Z"] for x in sts], [x["dX"] for x in sts],
                                       None if f == 1 else [L["dU"] for L in Ls], None if f == 2 else [L["dV"] for L in Ls],
                                       None if f == 1 else [L["db"] for L in Ls], f, [L["ws"] for L in Ls])

        def one_fwd(L, s, f):
            st = L["sets"][s]
            b.lrd_linear_fwd(L["desc"], st["X"], L["V"], L["U"], L["b"], st["Y"], None if f == 1 else st["Z"], f, L["ws"])

        def one_bwd(L, s, f):
            st = L["sets"][s]
            b.lrd_linear_bwd(L["desc"], st["dY"], None if f == 2 else st["X"], L["V"], L["U"], None if f == 1 else st["Z"], st["dX"],
                             None if f == 1 else L["dU"], None if f == 2 else L["dV"], None if f == 1 else L["db"], f, L["ws"])

        def lrd_stack(s, f):
            # the q / k / v workspaces are shared by the blocks' groups, which follow one another in the stream
            for bi, layers in enumerate(blocks):
                ss = (s + bi) % S
                g_call(layers[:3], ss, f, True)
                for L in layers[3:]:
                    one_fwd(L, ss, f)
            for bi, layers in reversed(list(enumerate(blocks))):
                ss = (s + bi) % S
                for L in reversed(layers[3:]):
                    if args.wgrad != "beside":
                        one_bwd(L, ss, f)
                        continue
                    # the weight gradients on a second stream beside the next layer's data pass (each layer of each
                    # block has its own workspace: the weights call reads the dZ its data call left there)
                    st = L["sets"][ss]
                    cur = torch.cuda.current_stream()
                    b.lrd_linear_bwd_data(L["desc"], st["dY"], L["V"], L["U"], st["dX"], f, L["ws"])
                    c4_w.wait_stream(cur)
                    with torch.cuda.stream(c4_w):
                        b.lrd_linear_bwd_weights(L["desc"], st["dY"], None if f == 2 else st["X"], None if f == 1 else st["Z"],
                                                 None if f == 1 else L["dU"], None if f == 2 else L["dV"], None if f == 1 else L["db"], f, L["ws"])
                g_call(layers[:3], ss, f, False)
            if args.wgrad == "beside":
                torch.cuda.current_stream().wait_stream(c4_w)

        c4_w = torch.cuda.Stream()

        def dense_stack(s):
            for bi, layers in enumerate(blocks):
                for L in layers:
                    st = L["sets"][(s + bi) % S]
                    b.lrd_dense_fwd(L["ddesc"], st["X"], L["W"], L["b"], st["Y"], L["wsd"])
            for bi, layers in reversed(list(enumerate(blocks))):
                for L in reversed(layers):
                    st = L["sets"][(s + bi) % S]
                    b.lrd_dense_bwd(L["ddesc"], st["dY"], st["X"], L["W"], st["dX"], L["dW"], L["db"], L["wsd"])

        def stack_work(f):
            fl = by = t = 0.0
            for name, K, N, r in wl.C4_GPT_LAYERS:
                for which in ("fwd", "bwd"):
                    a_, c_ = layer_flops(M, K, N, r, f, which), layer_bytes(M, K, N, r, f, which)
                    fl += a_ * NB
                    by += c_ * NB
                    t += NB * max(a_ / (peaks["bf16_tflops"] * 1e12), c_ / (peaks["hbm_gbs"] * 1e9))
            return fl, by, t
        res = {}
        for f, label in ((1, "U frozen (phase 0)"), (2, "V frozen (phase 1)"), (0, "nothing frozen")):
            sec, spread = time_graph(torch, lambda s, f=f: lrd_stack(s, f), S, reps=max(2, reps // 2))
            fl, by, t = stack_work(f)
            res[f] = (sec, spread, fl, t)
            variants.append({"variant": label, "ms": sec * 1e3, "tokens_per_s": M / sec, "tflops": fl / sec / 1e12, "frac": t / sec,
                             "kernels": count(lambda: lrd_stack(0, f))})
        sec, spread = time_graph(torch, dense_stack, S, reps=max(2, reps // 2))
        fl = t = 0.0
        for name, K, N, r in wl.C4_GPT_LAYERS:
            a_, c_ = dense_flops_bytes(M, K, N)
            fl += a_ * NB
            t += NB * max(a_ / (peaks["bf16_tflops"] * 1e12), c_ / (peaks["hbm_gbs"] * 1e9))
        variants.append({"variant": "undecomposed stack", "ms": sec * 1e3, "tokens_per_s": M / sec, "tflops": fl / sec / 1e12, "frac": t / sec,
                         "kernels": count(lambda: dense_stack(0))})
        sec = 0.5 * (res[1][0] + res[2][0])
        spread = (min(res[1][1][0], res[2][1][0]), max(res[1][1][1], res[2][1][1]))
        fl, t = 0.5 * (res[1][2] + res[2][2]), 0.5 * (res[1][3] + res[2][3])
        roof = {"bound": "tensor", "achieved": fl / sec / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": t / sec, "traffic": None,
                "note": "frac = sum over layers of max(flops at the tensor peak, bytes at the HBM peak) / time; achieved = useful TFLOP/s"}
        h2d = [(L["sets"][0]["X"], L["hX"]) for L in blocks[0]] + [(L["sets"][0]["dY"], L["hdY"]) for L in blocks[0]]
        d2h = [(L["hdV"], L["dV"]) for L in blocks[0]]
        e2e_t = time_e2e(torch, lambda: lrd_stack(0, 1), h2d, d2h, max(2, args.steps // 10))
        cpu = None
        if want_cpu:
            Ms = 512
            ccs = []
            for i, (name, K, N, r) in enumerate(wl.C4_GPT_LAYERS):
                cc = wl.random_factor_case(Ms, K, N, r, "bf16", 4100 + i)
                ccs.append({k: cc[k].astype(np.float64) for k in ("X", "V", "U", "b", "dY")})

            def cpu_step():
                for cc in ccs:
                    Z, _ = o.linear_fwd(cc["X"], cc["V"], cc["U"], cc["b"])
                    o.linear_bwd(cc["dY"], cc["X"], cc["V"], cc["U"], Z, 1)
            csec, creps = time_oracle(cpu_step, 8.0)
            cpu = {"value": Ms / (csec * NB), "unit": "tokens/s", "cores": threads, "kind": "oracle",
                   "sample": f"scaled: {creps} x one block's six layers (U frozen) on a slice of {Ms} of the {M} tokens, times {NB} blocks"}
        nk = (variants[0]["kernels"] + variants[1]["kernels"]) // 2
        return finish("c4", "configs[4]: the LRD linear layers of a 12-block GPT-2-medium-shaped stack (hidden 1024, FFN 4096, r=256 attention / r=512 FFN), "
                      "M=8192 tokens, bf16, fwd through all blocks then bwd in reverse; mean of the two phases of sequential freezing (U frozen, V frozen); "
                      "layer norm, attention, GELU, embedding and loss are not part of the method and do not run", M, sec, spread, "bf16", roof, cpu, e2e_t,
                      nk * args.steps, {"l2": f"cycling {S} activation buffer sets per layer (1.3 GB)", "h2d": "one block's activations per step (the stack's layers share them)"})
    raise SystemExit(f"unknown config {args.config}")


# ---- our arm ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c1", choices=["c0", "c1", "c2", "c3", "c4"], help="workload (default: the BERT-base-shaped block)")
    ap.add_argument("--sets", type=int, default=4, help="distinct activation buffer sets cycled through (L2 eviction)")
    ap.add_argument("--path", default="auto", choices=["auto", "general", "unfused", "fused"])
    ap.add_argument("--groups", default="qkv", choices=["none", "qkv"],
                    help="qkv: the three independent attention projections go out as one group (the default); none: one call per layer")
    ap.add_argument("--wgrad", default="beside", choices=["beside", "inline"],
                    help="beside: a layer's weight gradients run on a second stream beside the next layer's data pass (lrd_linear_bwd_data + "
                         "lrd_linear_bwd_weights; the step ends when both streams have finished); inline: one lrd_linear_bwd call per layer")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch through the C ABI every step instead of CUDA graphs")
    ap.add_argument("--single-step-graphs", action="store_true", help="one CUDA graph per step instead of one per cycle of steps (every buffer set under both masks)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.config != "c1":
        return run_other(args)

    import torch
    import torch.distributed as dist
    from paper_2309_03824_b200 import build as lrd_build
    lrd_build.build()
    from paper_2309_03824_b200 import binding as b
    from paper_2309_03824_b200 import decompose
    from paper_2309_03824_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU path exists)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peak_src = load_peaks()
    b.lrd_set_path({"auto": 0, "general": 1, "unfused": 2, "fused": 3}[args.path])
    args.warmup = max(args.warmup, 3)
    args.steps += args.steps % 2                    # both masks equally often
    bf = torch.bfloat16

    # ---- inputs: seeded on the host, one rounding to bf16, then resident on the device -------------
    cases = make_layers_numpy(decompose.svd_factors)
    S = max(1, args.sets)
    layers = []
    act_bytes_per_set = 0
    for c in cases:
        M, K, N, r = c["M"], c["K"], c["N"], c["r"]
        L = {"name": c["name"], "M": M, "K": K, "N": N, "r": r, "desc": b.linear_desc(M, K, N, r, b.LRD_BF16)}
        L["V"], L["U"], L["b"] = (torch.from_numpy(c[k]).to("cuda", bf) for k in ("V", "U", "b"))
        L["hX"] = torch.from_numpy(c["X"]).to(bf).pin_memory()
        L["hdY"] = torch.from_numpy(c["dY"]).to(bf).pin_memory()
        L["sets"] = []
        for s in range(S):
            st = {"X": L["hX"].to("cuda"), "dY": L["hdY"].to("cuda"),
                  "Y": torch.empty(M, N, dtype=bf, device="cuda"), "Z": torch.empty(M, r, dtype=bf, device="cuda"),
                  "dX": torch.empty(M, K, dtype=bf, device="cuda")}
            L["sets"].append(st)
        act_bytes_per_set += 2 * 2 * (M * K + M * N) + 2 * M * r
        L["dU"] = torch.empty(N, r, dtype=bf, device="cuda")
        L["dV"] = torch.empty(K, r, dtype=bf, device="cuda")
        L["db"] = torch.empty(N, dtype=bf, device="cuda")
        L["hdU"] = torch.empty(N, r, dtype=bf).pin_memory()
        L["hdV"] = torch.empty(K, r, dtype=bf).pin_memory()
        L["hdb"] = torch.empty(N, dtype=bf).pin_memory()
        nws = max(b.lrd_linear_workspace_bytes(L["desc"], 0, 0), b.lrd_linear_workspace_bytes(L["desc"], 0, 1), 256)
        L["ws"] = torch.empty(nws, dtype=torch.uint8, device="cuda")
        layers.append(L)

    def fwd(L, st, freeze):
        b.lrd_linear_fwd(L["desc"], st["X"], L["V"], L["U"], L["b"], st["Y"], None if freeze == b.LRD_FREEZE_U else st["Z"],
                         freeze, L["ws"])

    def bwd(L, st, freeze):
        b.lrd_linear_bwd(L["desc"], st["dY"], None if freeze == b.LRD_FREEZE_V else st["X"], L["V"], L["U"],
                         None if freeze == b.LRD_FREEZE_U else st["Z"], st["dX"],
                         None if freeze == b.LRD_FREEZE_U else L["dU"], None if freeze == b.LRD_FREEZE_V else L["dV"],
                         None if freeze == b.LRD_FREEZE_U else L["db"], freeze, L["ws"])

    # The query, key and value projections of a block depend on nothing the others produce: they go out as one
    # group (side by side); the output projection and the two feed-forward layers follow one another.
    group = [L for L in layers if L["name"] in ("attn_q", "attn_k", "attn_v")] if args.groups != "none" else []
    singles = [L for L in layers if not any(L is G for G in group)]

    def group_fwd(Ls, s, freeze):
        sts = [L["sets"][s] for L in Ls]
        b.lrd_linear_group_fwd([L["desc"] for L in Ls], [st["X"] for st in sts], [L["V"] for L in Ls], [L["U"] for L in Ls],
                               [L["b"] for L in Ls], [st["Y"] for st in sts],
                               None if freeze == b.LRD_FREEZE_U else [st["Z"] for st in sts], freeze, [L["ws"] for L in Ls])

    def group_bwd(Ls, s, freeze):
        sts = [L["sets"][s] for L in Ls]
        fu, fv = freeze == b.LRD_FREEZE_U, freeze == b.LRD_FREEZE_V
        b.lrd_linear_group_bwd([L["desc"] for L in Ls], [st["dY"] for st in sts], None if fv else [st["X"] for st in sts],
                               [L["V"] for L in Ls], [L["U"] for L in Ls], None if fu else [st["Z"] for st in sts],
                               [st["dX"] for st in sts], None if fu else [L["dU"] for L in Ls], None if fv else [L["dV"] for L in Ls],
                               None if fu else [L["db"] for L in Ls], freeze, [L["ws"] for L in Ls])

    def bwd_data(L, st, freeze):
        b.lrd_linear_bwd_data(L["desc"], st["dY"], L["V"], L["U"], st["dX"], freeze, L["ws"])

    def bwd_weights(L, st, freeze):
        b.lrd_linear_bwd_weights(L["desc"], st["dY"], None if freeze == b.LRD_FREEZE_V else st["X"], None if freeze == b.LRD_FREEZE_U else st["Z"],
                                 None if freeze == b.LRD_FREEZE_U else L["dU"], None if freeze == b.LRD_FREEZE_V else L["dV"],
                                 None if freeze == b.LRD_FREEZE_U else L["db"], freeze, L["ws"])

    # Nothing later in the backward pass waits for a layer's weight gradients: with --wgrad beside they go to a second
    # stream (lower priority than the data pass) and run beside the next layer's data pass on the SMs that pass leaves
    # idle; the step ends when both streams are done.
    w_stream = torch.cuda.Stream() if args.wgrad == "beside" else None

    def step_eager(s, freeze):
        if group:
            group_fwd(group, s, freeze)
        for L in singles:
            fwd(L, L["sets"][s], freeze)
        cur_s = torch.cuda.current_stream()
        for L in reversed(singles):
            if w_stream is None:
                bwd(L, L["sets"][s], freeze)
                continue
            bwd_data(L, L["sets"][s], freeze)
            w_stream.wait_stream(cur_s)
            with torch.cuda.stream(w_stream):
                bwd_weights(L, L["sets"][s], freeze)
        if group:
            group_bwd(group, s, freeze)
        if w_stream is not None:
            cur_s.wait_stream(w_stream)

    masks = [b.LRD_FREEZE_U, b.LRD_FREEZE_V]
    # warm every (set, mask) once outside any capture: one-time kernel attribute set-up happens here
    for s in range(S):
        for f in masks:
            step_eager(s, f)
    torch.cuda.synchronize()
    if b.lrd_check_device_status() != b.LRD_OK:
        raise SystemExit("device-side wait timed out during warm-up")
    n0 = b.lrd_launch_count()
    step_eager(0, masks[0])
    step_eager(0, masks[1])
    launches_per_two_steps = b.lrd_launch_count() - n0

    graphs = {}
    if not args.no_graph:
        side = torch.cuda.Stream(priority=-1)
        for s in range(S):
            for f in masks:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(g, stream=side):
                        step_eager(s, f)
                graphs[(s, f)] = g
        torch.cuda.synchronize()

    # One graph for a whole cycle of steps (every buffer set once, under both masks = 2 S steps): the dependent-launch
    # overlap then also holds across step boundaries, and the cost of a graph launch (about 10 us of device idle time
    # between two replays) is paid once per cycle.  Steps that do not fill a cycle replay the single-step graphs.
    cycle = 2 * S
    cycle_graph = None
    if graphs and not args.single_step_graphs:
        side = torch.cuda.Stream(priority=-1)
        cycle_graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(cycle_graph, stream=side):
                for s in range(S):
                    step_eager(s, masks[0])
                    step_eager(s, masks[1])
        torch.cuda.synchronize()

    def step(i):
        s, f = (i // 2) % S, masks[i % 2]
        if graphs:
            graphs[(s, f)].replay()
        else:
            step_eager(s, f)

    def run_steps(start, n):
        """Steps start .. start + n - 1, exactly n of them."""
        i, end = start, start + n
        while i < end:
            if cycle_graph is not None and i % cycle == 0 and i + cycle <= end:
                cycle_graph.replay()
                i += cycle
            else:
                step(i)
                i += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, bulk=False):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        if bulk:
            fn(0, steps)
        else:
            for i in range(steps):
                fn(i)
        e1.record()
        torch.cuda.synchronize()
        t1 = time.time()
        ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        barrier()
        return ms, t0, t1

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        t_wait = time.time()
        while not sampler.rows and time.time() - t_wait < 5.0:      # nvidia-smi takes a moment to print its first sample
            time.sleep(0.05)
    if cycle_graph is not None:           # the cycle graph's first replay (which uploads it) stays outside the timed region
        cycle_graph.replay()              # whatever --warmup is
    run_steps(0, args.warmup)
    # the timed region (exactly --steps steps) is taken five times; the median is reported, the spread beside it
    samples = []
    t0 = t1 = None
    for _ in range(5):
        ms_i, a0, a1 = timed(run_steps, args.steps, bulk=True)
        samples.append(ms_i)
        t0, t1 = (a0 if t0 is None else t0), a1
    samples.sort()
    ms = samples[len(samples) // 2]
    # The timed region is shorter than one sampling period (K steps of ~0.2 ms): the same steps go on, untimed, for
    # about a second and a half so that the clock samples are taken under this very load.
    if rank == 0:
        i = args.steps
        while time.time() - t1 < 1.5:
            run_steps(i, 12 * cycle)
            i += 12 * cycle
            torch.cuda.synchronize()
    barrier()
    clocks = sampler.summary(t0, time.time()) if rank == 0 else None
    ms_per_step = ms / args.steps
    # the same steps on ONE buffer set (its 239 MB partly stay in L2 from step to step): reported beside the headline, labelled
    hot = None
    if S > 1:
        hot_graph = None
        if cycle_graph is not None:              # the same cycle of 2 S steps, all on buffer set 0
            side = torch.cuda.Stream(priority=-1)
            hot_graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(hot_graph, stream=side):
                    for _ in range(S):
                        step_eager(0, masks[0])
                        step_eager(0, masks[1])
            torch.cuda.synchronize()

        def hot_steps_run(start, n):
            i, end = start, start + n
            while i < end:
                if hot_graph is not None and i % cycle == 0 and i + cycle <= end:
                    hot_graph.replay()
                    i += cycle
                else:
                    f = masks[i % 2]
                    if graphs:
                        graphs[(0, f)].replay()
                    else:
                        step_eager(0, f)
                    i += 1
        hot_steps_run(0, cycle)
        hot_steps = max(2, min(args.steps, 200) // 2 * 2)
        hms, _, _ = timed(hot_steps_run, hot_steps, bulk=True)
        hot = {"ms_per_step": hms / hot_steps, "steps": hot_steps,
               "note": "one activation buffer set re-used every step (partly L2-resident); not the headline"}
    tokens = wl.C1_M * world
    value = whole_job_value(wl.C1_M, world, ms_per_step)

    # ---- end to end: activations from pinned host memory in, weight gradients out, every step ------
    h2d = sum(L["hX"].numel() * 2 + L["hdY"].numel() * 2 for L in layers)

    def d2h_bytes(f):
        return sum(((L["N"] * L["r"] + L["N"]) if f != b.LRD_FREEZE_U else 0) * 2 + ((L["K"] * L["r"]) if f != b.LRD_FREEZE_V else 0) * 2
                   for L in layers)

    # Three streams: the inputs of step i + 1 cross PCIe while step i computes; the gradients leave on a third
    # stream, and the next step's kernels wait for them (the gradient buffers are shared by all sets).  Every
    # step's copies are enqueued inside the timed region; with a single buffer set the step runs serially.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(S)]
    ev_comp = [None] * S
    issued = set()
    e2e_last = [0]

    def e2e_copy_in(i):
        if i in issued:
            return
        issued.add(i)
        s = i % S
        if ev_comp[s] is not None:
            s_in.wait_event(ev_comp[s])          # the set's previous user has finished computing
        with torch.cuda.stream(s_in):
            for L in layers:
                L["sets"][s]["X"].copy_(L["hX"], non_blocking=True)
                L["sets"][s]["dY"].copy_(L["hdY"], non_blocking=True)
            ev_in[s].record(s_in)

    def e2e_step(i):
        s, f = i % S, masks[i % 2]
        if S == 1:
            for L in layers:
                L["sets"][0]["X"].copy_(L["hX"], non_blocking=True)
                L["sets"][0]["dY"].copy_(L["hdY"], non_blocking=True)
        else:
            e2e_copy_in(i)
            if i + 1 < e2e_last[0]:
                e2e_copy_in(i + 1)
            cur.wait_event(ev_in[s])
        if graphs:
            graphs[(s, f)].replay()
        else:
            step_eager(s, f)
        if S > 1:
            ev_comp[s] = torch.cuda.Event()
            ev_comp[s].record(cur)
            s_out.wait_event(ev_comp[s])
        with torch.cuda.stream(s_out if S > 1 else cur):
            for L in layers:
                if f != b.LRD_FREEZE_U:
                    L["hdU"].copy_(L["dU"], non_blocking=True)
                    L["hdb"].copy_(L["db"], non_blocking=True)
                if f != b.LRD_FREEZE_V:
                    L["hdV"].copy_(L["dV"], non_blocking=True)
        if S > 1:
            cur.wait_stream(s_out)               # the step ends when its result is on the host

    e2e_steps = max(4, min(args.steps, 40))
    e2e_steps += e2e_steps % 2
    e2e_last[0] = 4
    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    issued.clear()
    e2e_last[0] = e2e_steps
    ems, _, _ = timed(e2e_step, e2e_steps)
    e2e_val = tokens / (ems / e2e_steps * 1e-3)
    d2h = (d2h_bytes(masks[0]) + d2h_bytes(masks[1])) // 2

    # ---- the dominant kernel alone: the fused forward chain of the widest layer (one launch per call) --
    roof = None
    kernels = []
    if rank == 0:
        reps, rounds = 10, 8          # 10 replays of a graph of 8 x S launches of the op

        def time_op(fn):
            for s in range(S):
                fn(s)
            torch.cuda.synchronize()
            n_before = b.lrd_launch_count()
            fn(0)
            n_k = b.lrd_launch_count() - n_before
            side2 = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side2):
                with torch.cuda.graph(g, stream=side2):
                    for _ in range(rounds):          # many launches per graph: a graph launch costs ~14 us of idle device
                        for s in range(S):
                            fn(s)
            torch.cuda.synchronize()
            g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e-3 / (reps * rounds * S), n_k

        for L in layers[3:]:          # one attention layer and both FFN layers
            M, K, N, r = L["M"], L["K"], L["N"], L["r"]
            for which, f in (("fwd", b.LRD_FREEZE_U), ("bwd", b.LRD_FREEZE_U), ("bwd", b.LRD_FREEZE_V)):
                if which == "fwd":
                    sec, nk = time_op(lambda s, L=L, f=f: fwd(L, L["sets"][s], f))
                else:
                    sec, nk = time_op(lambda s, L=L, f=f: bwd(L, L["sets"][s], f))
                fl, by = layer_flops(M, K, N, r, f, which), layer_bytes(M, K, N, r, f, which)
                t_t, t_h = fl / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)
                kernels.append({"op": f"{L['name']} {which} freeze={'U' if f == 1 else 'V'}", "kernels": nk,
                                "us": sec * 1e6, "tflops": fl / sec / 1e12, "gbs": by / sec / 1e9,
                                "bound": "tensor" if t_t >= t_h else "hbm", "frac": max(t_t, t_h) / sec})
        dom = next(k for k in kernels if k["op"].startswith("ffn_1 fwd"))
        if dom["bound"] == "tensor":
            roof = {"bound": "tensor", "achieved": dom["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": dom["tflops"] / peaks["bf16_tflops"]}
        else:
            roof = {"bound": "hbm", "achieved": dom["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": dom["gbs"] / peaks["hbm_gbs"]}
        fresh = kernel_digest() == NCU_TRAFFIC["digest"]
        worst = min(kernels, key=lambda k: k["frac"])
        roof.update({"traffic": NCU_TRAFFIC["bytes_per_launch"] if fresh else None,
                     "traffic_note": NCU_TRAFFIC["note"] if fresh else "no counters for the kernel as it is now",
                     "l2_to_sm_bytes": NCU_TRAFFIC["l2_to_sm_bytes_per_launch"] if fresh else None,
                     "kernel": dom["op"], "kernels_in_op": dom["kernels"], "peak_source": peak_src, "us_per_launch": dom["us"],
                     "worst_op": {"op": worst["op"], "frac": worst["frac"], "bound": worst["bound"], "us": worst["us"]},
                     "time_weighted_frac_of_timed_ops": sum(k["frac"] * k["us"] for k in kernels) / sum(k["us"] for k in kernels)})
        for k in kernels:
            log(json.dumps(k))

    # ---- whole-step roofline (the slower of flops at the tensor peak and bytes at the HBM peak) -------
    step_roof = {}
    for f in masks:
        t = 0.0
        for L in layers:
            for which in ("fwd", "bwd"):
                t += max(layer_flops(L["M"], L["K"], L["N"], L["r"], f, which) / (peaks["bf16_tflops"] * 1e12),
                         layer_bytes(L["M"], L["K"], L["N"], L["r"], f, which) / (peaks["hbm_gbs"] * 1e9))
        step_roof[f] = t
    t_roof = 0.5 * (step_roof[masks[0]] + step_roof[masks[1]])
    useful_flops = 0.5 * sum(layer_flops(L["M"], L["K"], L["N"], L["r"], f, "both") for L in layers for f in masks)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        np_cases = [{k: (c[k].astype(np.float64) if isinstance(c[k], np.ndarray) else c[k]) for k in c} for c in cases]
        sec, reps_c, threads = oracle_block_seconds(np_cases, 10.0)
        cpu = {"value": wl.C1_M / sec, "unit": "tokens/s", "cores": threads, "kind": "oracle",
               "sample": f"{reps_c} full steps of the same block at M=4096, masks alternating ({sec * reps_c:.1f} s of CPU work)"}
    if rank == 0:
        sampler.stop()
        line = {"metric": "LRD layer fwd+bwd tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": config_dict({"parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                                       "l2": f"cycling {S} activation buffer sets, {S * act_bytes_per_set / 1e6:.0f} MB > 126 MB L2",
                                       "launch": "eager C-ABI calls" if args.no_graph else ("CUDA graph replay of the C-ABI calls, one graph per step" if args.single_step_graphs
                                                  else f"CUDA graph replay of the C-ABI calls, one graph per cycle of {cycle} steps (every buffer set under both masks)"),
                                       "path": args.path,
                                       "weight_gradients": {"beside": "on a second stream beside the next layer's data pass (two-call backward), joined at the end of the step",
                                                            "inline": "one backward call per layer"}[args.wgrad],
                                       "groups": {"qkv": "attn_q/k/v side by side in one group call, the other layers one call each",
                                                  "none": "one call per layer"}[args.groups]}),
                "repeats": {"n": len(samples), "min_ms": samples[0] / args.steps, "max_ms": samples[-1] / args.steps, "reported": "median"},
                "useful_tflops": useful_flops * world / (ms_per_step * 1e-3) / 1e12,
                "step_roofline_frac": t_roof / (ms_per_step * 1e-3), "step_roofline_us": t_roof * 1e6,
                "roofline": roof, "hot_cache": hot, "cpu_baseline": cpu,
                "e2e": {"value": e2e_val, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
                "gpu_launches": int(launches_per_two_steps * args.steps // 2), "clocks": clocks, "peaks": peak_src}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
