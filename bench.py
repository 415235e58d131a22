#!/usr/bin/env python
"""Benchmark of the decomposed-layer training step on B200.

Default workload: the BERT-base-shaped block (four 768->768 layers at r=192, 768->3072 and
3072->768 at r=384, M = 4096 tokens, bf16 with fp32 accumulation), forward + backward of every
layer per step, sequential freezing alternating U-frozen / V-frozen every step.

One JSON line on stdout (rank 0).  `value` is tokens/s with inputs resident in HBM; `e2e` is the
same step with the activations copied from pinned host memory and the weight gradients copied
back inside the timed region; `roofline` is the dominant kernel, timed alone with CUDA events;
`cpu_baseline` is the fp64 CPU oracle timed on this machine's host cores.
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
NCU_TRAFFIC = {"digest": "4ada81cd16d2e7b7", "bytes_per_launch": 9319168}
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


# ---- our arm ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sets", type=int, default=4, help="distinct activation buffer sets cycled through (L2 eviction)")
    ap.add_argument("--path", default="auto", choices=["auto", "general", "unfused", "fused"])
    ap.add_argument("--groups", default="qkv", choices=["none", "qkv"],
                    help="qkv: the three independent attention projections go out as one group (the default); none: one call per layer")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch through the C ABI every step instead of CUDA graphs")
    ap.add_argument("--single-step-graphs", action="store_true", help="one CUDA graph per step instead of one per cycle of steps (every buffer set under both masks)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

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

    def step_eager(s, freeze):
        if group:
            group_fwd(group, s, freeze)
        for L in singles:
            fwd(L, L["sets"][s], freeze)
        for L in reversed(singles):
            bwd(L, L["sets"][s], freeze)
        if group:
            group_bwd(group, s, freeze)

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
        side = torch.cuda.Stream()
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
        side = torch.cuda.Stream()
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
    run_steps(0, args.warmup)
    ms, t0, t1 = timed(run_steps, args.steps, bulk=True)
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
            side = torch.cuda.Stream()
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
        traffic = NCU_TRAFFIC["bytes_per_launch"] if kernel_digest() == NCU_TRAFFIC["digest"] else None
        roof.update({"traffic": traffic, "kernel": dom["op"], "kernels_in_op": dom["kernels"], "peak_source": peak_src,
                     "us_per_launch": dom["us"]})
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
                                       "groups": {"qkv": "attn_q/k/v side by side in one group call, the other layers one call each",
                                                  "none": "one call per layer"}[args.groups]}),
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
