#!/usr/bin/env python
"""Benchmark of the tile-hybrid linear layer (hybrid dense / 2:4 tile GEMM) on B200.

One step = one pass of the hot path over one batch of synthetic input: every GEMM of the
workload's case list, launched back to back from one CUDA graph (the paper times generation
through CUDA graphs as well).  Default workload: the LLaMA-2-7B-shaped decode linears
(3 weight shapes x 2:4-tile fraction in {0, .35, .7, 1} x M in {1, 16} = 24 GEMMs over 12
packed matrices, ~0.66 GB of packed weights per pass, so every weight read comes from HBM).

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_23410_b200 import inputs  # noqa: E402

HBM_SPEC_GBS = 8000.0            # roofline constants of the task definition
DENSE_SPEC_TFLOPS = 2250.0
SPARSE_SPEC_TFLOPS = 4500.0
L2_BYTES = 126e6


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def workload_cases(name: str, stack_m: int = 1):
    if name == "decode":
        cases = inputs.decode_cases()
        # all M=1 GEMMs first, then all M=16: a matrix is re-read only after ~0.66 GB of other weights
        return sorted(cases, key=lambda c: c["M"])
    if name == "decode-q4":
        return sorted(inputs.decode_q4_cases(), key=lambda c: c["M"])
    if name == "prefill":
        return sorted(inputs.prefill_cases(), key=lambda c: c["M"])
    if name == "13b":
        return sorted(inputs.llama13b_cases(), key=lambda c: c["M"])
    if name == "single":
        return [inputs.single_gemm_case()]
    if name == "stack":
        # 32 blocks x (q,k,v,o,gate,up,down) = 224 matrices, per-matrix 2:4-tile fraction ~ U[0,1]
        return [dict(c, M=stack_m) for c in inputs.stack_cases()]
    if name == "stack-fused":
        # the same weights with q/k/v and gate/up stored as one matrix each: 128 GEMMs
        return [dict(c, M=stack_m) for c in inputs.stack_fused_cases()]
    raise SystemExit(f"unknown workload {name}")


def case_costs(case, layout):
    """Algorithmic bytes and flops of one GEMM (realised tile counts, not expected ones)."""
    M, N, K = case["M"], case["N"], case["K"]
    T = (N // 128) * (K // 128)
    nbytes = layout.payload_bytes + 16 * T + M * K * 2 + M * N * 2
    f_dense = 2.0 * M * 16384 * (layout.n_dense + layout.n_dense_q4)
    f_sparse = 2.0 * M * 16384 * (layout.n_sparse + layout.n_sparse_q4)
    return dict(bytes=float(nbytes), flops=f_dense + f_sparse, f_dense=f_dense, f_sparse=f_sparse)


def roofline_seconds(cost, hbm_gbs, dense_tf, sparse_tf):
    t_mem = cost["bytes"] / (hbm_gbs * 1e9)
    t_tc = cost["f_dense"] / (dense_tf * 1e12) + cost["f_sparse"] / (sparse_tf * 1e12)
    return max(t_mem, t_tc), ("hbm" if t_mem >= t_tc else "tensor")


# ---------------------------------------------------------------------------------------------
# clocks sampler


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.samples = []
        self.proc = None
        self.index = index
        self.marks = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.12)
        self.proc.terminate()
        rows = [s for t, s in self.samples if t0 - 0.05 <= t <= t1 + 0.1] or [s for _, s in self.samples[-3:]]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); smax.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores


def oracle_sample(cases, budget_s):
    """Time the oracle GEMM on the leading cases of the step until ~budget_s of CPU work."""
    import oracle
    oracle.build()
    done, flops, secs, passes = [], 0.0, 0.0, 0
    prepared = {}
    while secs < budget_s and passes < 64:
        for case in cases:
            key = case["name"]
            if key not in prepared:
                if passes > 0:
                    continue
                W, flags, X = inputs.make_case_inputs(case)
                prepared[key] = (X, oracle.prune(W, flags))
            X, What = prepared[key]
            t = time.perf_counter()
            oracle.gemm_f64(X, What, want_bf16=True)
            secs += time.perf_counter() - t
            flops += 2.0 * case["M"] * case["N"] * case["K"]
            if passes == 0:
                done.append(key)
            if secs >= budget_s:
                break
        passes += 1
    # the oracle's pack (single-threaded C loops) on the first matrix, next to patch_pack's GB/s
    W, flags, _ = inputs.make_case_inputs(cases[0])
    t = time.perf_counter()
    blob, _ = oracle.pack(W, flags)
    t_pack = time.perf_counter() - t
    return dict(value=flops / secs / 1e12, unit="TFLOP/s", cores=oracle.num_threads(), kind="oracle",
                sample=f"oracle GEMM (double accumulation) over the step's first {len(done)} GEMMs "
                       f"({done[0]} .. {done[-1]}), repeated for {secs:.1f} s of CPU time",
                pack_gbs=(W.nbytes + blob.nbytes) / t_pack / 1e9, pack_sample=f"oracle pack of {cases[0]['name']}, one thread"), secs


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cases = workload_cases(args.workload)
    # bounded sample per step: the two GEMMs (M = 1 and 16) on the first 4096 x 4096 matrix with mixed tiles
    sample = [c for c in cases if c["N"] == 4096 and c["K"] == 4096 and 0 < c["p"] < 1][:1]
    sample += [c for c in cases if c["N"] == 4096 and c["K"] == 4096 and 0 < c["p"] < 1 and c["M"] != sample[0]["M"]][:1]
    prepared = []
    for c in sample:
        W, flags, X = inputs.make_case_inputs(c)
        prepared.append((X, oracle.prune(W, flags), 2.0 * c["M"] * c["N"] * c["K"]))
    steps = min(args.steps, 50)
    for _ in range(min(args.warmup, 3)):
        for X, What, _ in prepared:
            oracle.gemm_f64(X, What)
    t0 = time.perf_counter()
    for _ in range(steps):
        for X, What, _ in prepared:
            oracle.gemm_f64(X, What)
    dt = time.perf_counter() - t0
    flops = sum(f for _, _, f in prepared) * steps
    value = flops / dt / 1e12
    names = ", ".join(c["name"] for c in sample)
    cpu = dict(value=value, unit="TFLOP/s", cores=oracle.num_threads(), kind="oracle",
               sample=f"{steps} steps of the oracle GEMM on {names}")
    print(json.dumps({
        "impl": "reference", "metric": "hybrid_tile_gemm_effective_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 3), "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_label(args), "sample": names},
        "cpu_baseline": cpu,
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------------------
# our arm: helpers shared by the headline workload and the prefill section


def launch_flags(B, mode):
    # weights are packed once, before any step; "independent": no GEMM of the step reads another GEMM's output, and
    # (third promise) every launch between two drains of the GPU writes an output buffer of its own -- see replicate()
    return B.WEIGHTS_STATIC | ((B.INPUT_STATIC | B.OUTPUT_STATIC) if mode == "independent" else 0)


def replicate(torch, js, n):
    """The job list n times over for one CUDA graph, every repetition with output buffers of its own: inside a graph
    consecutive launches overlap, and the output promise says that no launch of such a run touches another's Y.
    (Graph replays follow each other only after a full drain.)"""
    out = list(js)
    for _ in range(n - 1):
        out += [dict(j, Y=torch.empty_like(j["Y"])) for j in js]
    return out


def launch_all(B, js, mode, variant=0):
    for j in js:
        B.patch_gemm(j["X"], j["layout"], j["packed"], Y=j["Y"], workspace=j["ws"], variant=variant | launch_flags(B, mode))


def make_graph(torch, B, js, mode, variant=0):
    launch_all(B, js, mode, variant)        # first call sets kernel attributes; must precede capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        launch_all(B, js, mode, variant)
    return g


def time_graph(torch, g, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / reps


def per_case_table(torch, B, jobs, mode, peaks, variant=0):
    """Each GEMM on rotating copies of its packed weight (>= 3 x L2 of them), so that its weight reads come from HBM."""
    table = []
    for j in jobs:
        blob = j["packed"]
        n_copies = int(min(max(3 * L2_BYTES // blob.numel() + 1, 2), 24))
        copies = [blob.clone() for _ in range(n_copies)]
        js = [dict(j, packed=cp, Y=torch.empty_like(j["Y"])) for cp in copies]
        g = make_graph(torch, B, js, mode, variant)
        for _ in range(3):
            g.replay()
        t = time_graph(torch, g, 3) / n_copies
        # enough launches per graph (about 2 ms worth, at most 48 rounds) that the drain at its end does not show
        rounds = int(min(max(round(2e-3 / (t * n_copies)), 1), 48))
        if rounds > 1:
            g = make_graph(torch, B, replicate(torch, js, rounds), mode, variant)
            g.replay()
        t = time_graph(torch, g, 10) / (n_copies * rounds)
        rs, b = roofline_seconds(j["cost"], HBM_SPEC_GBS, DENSE_SPEC_TFLOPS, SPARSE_SPEC_TFLOPS)
        rm, _ = roofline_seconds(j["cost"], peaks["hbm_gbs"], peaks["bf16_tflops_sustained"],
                                 2 * peaks["bf16_tflops_sustained"])
        table.append(dict(name=j["case"]["name"], us=round(t * 1e6, 2),
                          eff_tflops=round(j["cost"]["flops"] / t / 1e12, 2), bound=b,
                          frac_spec=round(rs / t, 3), frac_measured=round(rm / t, 3),
                          f_sparse=round((j["layout"].n_sparse + j["layout"].n_sparse_q4) /
                                         ((j["layout"].N // 128) * (j["layout"].K // 128)), 3)))
        del copies, js, g
    return table


def speedup_table(table):
    """Speed-up of every hybrid / 2:4 case over the all-dense tile configuration of the same shape and M
    (the comparison the prefill workload asks for)."""
    dense = {}
    for c in table:
        if c["f_sparse"] == 0.0:
            dense[(c["name"].split(".p")[0], c["name"].rsplit(".M", 1)[1])] = c["us"]
    sp = []
    for c in table:
        base = dense.get((c["name"].split(".p")[0], c["name"].rsplit(".M", 1)[1]))
        if base and c["f_sparse"] > 0.0:
            # ceiling: 18 432 instead of 32 768 bytes per 2:4 tile where HBM binds, half the tensor time where the MMAs do
            ceiling = 1.0 / (1.0 - (0.4375 if c["bound"] == "hbm" else 0.5) * c["f_sparse"])
            sp.append(dict(name=c["name"], f_sparse=c["f_sparse"], speedup_vs_all_dense=round(base / c["us"], 3),
                           ceiling=round(ceiling, 3), bound=c["bound"]))
    return sp


def parity_check(torch, jobs, seed_rows=8):
    """`--check sampled`: the outputs the timed graph left behind against the oracle (rank 0, one GPU).  GEMMs of up to
    64 tokens are compared in full, larger ones on `seed_rows` token rows spread over the token tiles plus the first and
    the last row.  Returns the worst relative Frobenius error and the worst max |dY| / max |Yref| over the GEMMs."""
    import oracle
    oracle.build()
    to_bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    pruned, worst_f, worst_m, n_out = {}, 0.0, 0.0, 0
    for j in jobs:
        key = id(j["packed"])
        if key not in pruned:
            pruned[key] = oracle.prune(j["W_bits"]() if callable(j["W_bits"]) else j["W_bits"], j["flags"])
        What = pruned[key]
        M = j["case"]["M"]
        Xb, Yb = to_bits(j["X"]), to_bits(j["Y"])
        if M <= 64:
            ref, _ = oracle.gemm_f64(Xb, What)
            got = inputs.bf16_bits_to_f32(Yb)
        else:
            rows = np.unique(np.concatenate([np.linspace(0, M - 1, seed_rows).astype(np.int64), [0, M - 1]]))
            ref = oracle.gemm_f64_rows(Xb, rows, What)
            got = inputs.bf16_bits_to_f32(Yb[rows])
        relF, maxrel = oracle.parity_metrics(got, ref)
        worst_f, worst_m, n_out = max(worst_f, float(relF)), max(worst_m, float(maxrel)), n_out + ref.size
    return dict(relF=worst_f, maxrel=worst_m, gemms=len(jobs), outputs_compared=int(n_out),
                tolerance={"relF": 2e-3, "maxrel": 1e-2}, ok=bool(worst_f <= 2e-3 and worst_m <= 1e-2),
                how="timed graph's outputs vs the CPU oracle (double accumulation); M <= 64 in full, larger M on sampled token rows")


def prefill_section(args, torch, B, dev, peaks):
    """The tensor-core half of the metric on the default line: the 27 LLaMA-2-7B prefill GEMMs (3 shapes x
    M in {512, 2048, 4096} x 2:4-tile fraction in {0, .5, 1}) as one step from a CUDA graph.  Weights and activations
    are drawn on the device (torch Philox, seeded per matrix); the tile flags are the seeded Bernoulli draws of
    inputs.prefill_cases()."""
    cases = sorted(inputs.prefill_cases(), key=lambda c: c["M"])
    mats, xs, jobs = {}, {}, []
    for c in cases:
        key = (c["N"], c["K"], c["stream"])
        if key not in mats:
            gen = torch.Generator(device=dev)
            gen.manual_seed(inputs.MASTER_SEED * 1000 + 500 + len(mats))
            W = torch.empty((c["N"], c["K"]), dtype=torch.bfloat16, device=dev).normal_(0.0, 0.02, generator=gen)
            flags = inputs.case_flags(c)
            layout = B.patch_packed_size(c["N"], c["K"], flags)
            packed = torch.empty(layout.total_bytes, dtype=torch.uint8, device=dev)
            B.patch_pack(W, flags, layout=layout, out=packed)
            Wh = W.view(torch.int16).cpu().numpy().view(np.uint16) if args.check != "none" else None
            mats[key] = (layout, packed, flags, Wh)
            del W
        layout, packed, flags, Wh = mats[key]
        xkey = (c["M"], c["K"])
        if xkey not in xs:
            gen = torch.Generator(device=dev)
            gen.manual_seed(inputs.MASTER_SEED * 1000 + 900 + len(xs))
            xs[xkey] = torch.empty(xkey, dtype=torch.bfloat16, device=dev).normal_(0.0, 1.0, generator=gen)
        Y = torch.empty((c["M"], c["N"]), dtype=torch.bfloat16, device=dev)
        jobs.append(dict(case=c, layout=layout, packed=packed, X=xs[xkey], Y=Y, ws=None, cost=case_costs(c, layout),
                         W_bits=Wh, flags=flags))
    g = make_graph(torch, B, jobs, args.launch)
    # the step is power-capped: warm up until the clocks have settled (~0.3 s of back-to-back steps), then time
    steps, warm = max(3, min(100, args.steps)), max(3, min(100, args.steps))
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    sampler.start()
    for _ in range(warm):
        g.replay()
    torch.cuda.synchronize()
    t0 = time.time()
    step_s = time_graph(torch, g, steps)
    clocks = sampler.stop(t0, time.time())
    flops = sum(j["cost"]["flops"] for j in jobs)
    fd, fs = sum(j["cost"]["f_dense"] for j in jobs), sum(j["cost"]["f_sparse"] for j in jobs)
    sus = peaks["bf16_tflops_sustained"]
    peak_meas = (fd + fs) / (fd / sus + fs / (2 * sus))                 # flop-weighted mix, 2:4 tiles at twice the dense rate
    peak_spec = (fd + fs) / (fd / DENSE_SPEC_TFLOPS + fs / SPARSE_SPEC_TFLOPS)
    spec_t = sum(roofline_seconds(j["cost"], HBM_SPEC_GBS, DENSE_SPEC_TFLOPS, SPARSE_SPEC_TFLOPS)[0] for j in jobs)
    achieved = flops / step_s / 1e12
    out = {
        "workload": "llama2-7b prefill linears", "gemms_per_step": len(jobs), "steps": steps, "warmup": warm,
        "ms_per_step": step_s * 1e3, "value": achieved, "unit": "TFLOP/s", "launch": args.launch, "cuda_graph": True,
        "data": "synthetic (weights and activations drawn on the device)",
        "l2": "inputs larger than L2: a step streams 9 packed matrices (~0.5 GB) and 0.77 GB of outputs",
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak_meas, "unit": "TFLOP/s", "frac": achieved / peak_meas,
                     "frac_of_spec": spec_t / step_s, "peak_spec": peak_spec, "peak_source": peaks["source"] + " (sustained bf16; 2:4 tiles x2)",
                     "traffic": None,
                     "kernels": "prefill_pair_kernel (weights of one tile kind), prefill2_kernel / prefill_kernel (mixed weights, M = 512)"},
        "clocks": clocks,
        # the step is power-capped: its time times the sampled SM clock separates kernel changes from clock drift
        "ms_x_sm_ghz": step_s * 1e3 * (clocks.get("sm_mhz") or 0.0) / 1e3,
        "gpu_launches": steps * len(jobs),
    }
    table = per_case_table(torch, B, jobs, args.launch, peaks)
    out["cases"] = table
    out["speedup_vs_all_dense"] = speedup_table(table)
    if args.check != "none":
        g.replay()
        torch.cuda.synchronize()
        for j in jobs:
            j["ws"] = None
        out["parity"] = parity_check(torch, jobs)
    return out


# ---------------------------------------------------------------------------------------------
# our arm


def run_ours(args):
    import torch
    from paper_2509_23410_b200 import binding as B, replicas

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    B.lib()
    peaks = measured_peaks()

    def to_dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)

    cases = workload_cases(args.workload, args.stack_m)
    # ---- setup (untimed): weights, packing, activations; replicas: every rank holds the whole workload
    mats = {}
    pack_bytes, pack_secs, pack_dev_secs = 0.0, 0.0, 0.0
    for c in cases:
        key = (c["N"], c["K"], c["stream"])
        if key in mats:
            continue
        if args.workload.startswith("stack"):
            # 6.5 G weights: drawn on the device (torch Philox, seeded per matrix) instead of on the host
            gen = torch.Generator(device=dev)
            gen.manual_seed(inputs.MASTER_SEED * 1000 + len(mats))
            W = torch.empty((c["N"], c["K"]), dtype=torch.bfloat16, device=dev).normal_(0.0, 0.02, generator=gen)
        else:
            W = to_dev(inputs.weight(c["N"], c["K"], inputs.MASTER_SEED, *c["stream"]))
        flags = inputs.case_flags(c)
        layout = B.patch_packed_size(c["N"], c["K"], flags)
        packed = torch.empty(layout.total_bytes, dtype=torch.uint8, device=dev)
        B.patch_pack(W, flags, layout=layout, out=packed)          # warm
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.patch_pack(W, flags, layout=layout, out=packed)
        e1.record()
        torch.cuda.synchronize()
        pack_secs += e0.elapsed_time(e1) * 1e-3
        pack_bytes += c["N"] * c["K"] * 2 + layout.total_bytes
        # the same with the tile flags already on the device: no host work, header and table built by a kernel
        flags_dev = torch.from_numpy(np.ascontiguousarray(flags, dtype=np.uint8).reshape(-1)).to(dev)
        packed2 = torch.empty(layout.total_bytes, dtype=torch.uint8, device=dev)
        B.patch_pack_dev(W, flags_dev, out=packed2)                # warm
        e0.record()
        B.patch_pack_dev(W, flags_dev, out=packed2)
        e1.record()
        torch.cuda.synchronize()
        pack_dev_secs += e0.elapsed_time(e1) * 1e-3
        if not torch.equal(packed, packed2):
            raise SystemExit("patch_pack_dev and patch_pack disagree")
        keep_w = args.check != "none" and not args.workload.startswith("stack")
        mats[key] = (layout, packed, flags, inputs.weight(c["N"], c["K"], inputs.MASTER_SEED, *c["stream"]) if keep_w else None)
        del W, packed2
    jobs, stack_x, shared_ws = [], {}, {}
    for c in cases:
        layout, packed, flags, w_bits = mats[(c["N"], c["K"], c["stream"])]
        xkey = (c["M"], c["K"]) if args.workload.startswith("stack") else None
        if xkey is not None and xkey in stack_x:
            X = stack_x[xkey]                # the stack shares one activation per (M, K); outputs are not chained
        else:
            X = to_dev(inputs.activation(c["M"], c["K"], inputs.MASTER_SEED, *c["stream"], c["M"]))
            if xkey is not None:
                stack_x[xkey] = X
        Y = torch.empty((c["M"], c["N"]), dtype=torch.bfloat16, device=dev)
        wkey = (c["M"], c["N"])
        if wkey not in shared_ws:            # GEMMs on one stream are ordered, so they may share a workspace
            shared_ws[wkey] = torch.zeros(max(B.patch_gemm_workspace_size(layout, c["M"]), 256), dtype=torch.uint8, device=dev)
        ws = shared_ws[wkey]
        jobs.append(dict(case=c, layout=layout, packed=packed, X=X, Y=Y, ws=ws, cost=case_costs(c, layout),
                         W_bits=w_bits, flags=flags))
    weight_bytes = sum(m[0].total_bytes for m in mats.values())

    def mk_graph(js, mode=None):
        return make_graph(torch, B, js, mode or args.launch, args.variant)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def tm_graph(g, reps):
        return time_graph(torch, g, reps)

    step_graph = mk_graph(jobs)
    # several consecutive steps may be captured into one graph (a serving loop enqueues step after step on
    # one stream; a graph per step would end every step with a full drain that such a loop does not have)
    spg = max(1, min(args.steps_per_graph, args.steps))
    multi_graph = mk_graph(replicate(torch, jobs, spg)) if spg > 1 else step_graph
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step_graph.replay()
    if spg > 1:
        multi_graph.replay()
    barrier()
    t_wall0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps // spg):
        multi_graph.replay()
    for _ in range(args.steps % spg):
        step_graph.replay()
    e1.record()
    barrier()
    secs = e0.elapsed_time(e1) * 1e-3
    secs = replicas.max_over_ranks(secs, dev)
    step_s = secs / args.steps
    step_flops = sum(j["cost"]["flops"] for j in jobs)
    value = world * step_flops / step_s / 1e12

    # ---- spread: 50 more replays of the timed graph, each between its own pair of events (median and minimum;
    # every replay ends with a drain here, so these sit slightly above the back-to-back mean of the timed region)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(50)]
    for a, b in evs:
        a.record()
        multi_graph.replay()
        b.record()
    torch.cuda.synchronize()
    per_step = sorted(a.elapsed_time(b) / spg for a, b in evs)
    replay_stats = {"replays": len(per_step), "steps_per_replay": spg, "median_ms_per_step": per_step[len(per_step) // 2],
                    "min_ms_per_step": per_step[0], "max_ms_per_step": per_step[-1]}

    # ---- one step per graph replay, for comparison: every step then ends with a full drain of the GPU
    single_s = step_s
    if spg > 1:
        single_s = replicas.max_over_ranks(tm_graph(step_graph, max(10, args.steps // 5)), dev)

    # ---- the same step under the other launch promise (context for the headline number)
    other = "dependent" if args.launch == "independent" else "independent"
    g_other = mk_graph(replicate(torch, jobs, spg), other)
    for _ in range(3):
        g_other.replay()
    other_s = tm_graph(g_other, max(10, args.steps // 5 // spg)) / spg
    del g_other

    # ---- dominant kernel: the launches that take the largest share of the step, timed on their own
    groups = {}
    for j in jobs:
        groups.setdefault(j["case"]["M"], []).append(j)
    dom = None
    for M, js in groups.items():
        g = mk_graph(replicate(torch, js, spg))    # the same number of passes per graph as the timed step
        for _ in range(3):
            g.replay()
        t = tm_graph(g, max(10, args.steps // 10 // spg)) / spg
        if dom is None or t > dom[1]:
            dom = (M, t, js)
    dM, dt, djs = dom
    kernel_name = "decode_q4_kernel" if args.workload == "decode-q4" else B_kernel_name(dM, args.launch)
    bound = roofline_seconds(djs[0]["cost"], HBM_SPEC_GBS, DENSE_SPEC_TFLOPS, SPARSE_SPEC_TFLOPS)[1]
    per_launch = dt / len(djs)
    if bound == "hbm":
        alg = sum(j["cost"]["bytes"] for j in djs) / len(djs)
        achieved, peak, unit = alg / per_launch / 1e9, peaks["hbm_gbs"], "GB/s"
    else:
        alg = sum(j["cost"]["flops"] for j in djs) / len(djs)
        # mixed dense / sparse contraction: the peak is the flop-weighted mix (sparse tiles at twice the dense rate)
        fd = sum(j["cost"]["f_dense"] for j in djs)
        fs = sum(j["cost"]["f_sparse"] for j in djs)
        achieved, unit = alg / per_launch / 1e12, "TFLOP/s"
        peak = (fd + fs) / (fd / peaks["bf16_tflops_sustained"] + fs / (2 * peaks["bf16_tflops_sustained"]))
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    roof = dict(bound=bound, achieved=achieved, peak=peak, unit=unit, frac=achieved / peak,
                traffic=load_traffic(kernel_name, alg) if bound == "hbm" else None, kernel=kernel_name, launches_timed=len(djs),
                us_per_launch=per_launch * 1e6, peak_source=peaks["source"],
                algorithmic_per_launch=alg)
    if args.workload == "decode-q4":
        # HBM is the roof the bytes are counted against; the kernel's own ceiling is lower: every stored value costs
        # ~2 issue slots to dequantise (half-rate bf16x2 arithmetic among them), see the kernel's header
        roof["note"] = ("4-bit payloads: algorithmic bytes are 0.52 B (dense) / 0.39 B (2:4) per weight element; the kernel "
                        "dequantises into tensor memory and is bound by instruction issue before HBM")
        roof["frac_of_8tbs"] = achieved / HBM_SPEC_GBS
    elif bound == "hbm":
        roof["note"] = ("the measured peak is a copy (read + write) bandwidth; this kernel only reads, and a read-only "
                        "stream can exceed it (the ceiling is the 8 TB/s of frac_of_roofline_spec); ncu confirms that "
                        "every algorithmic byte is read from DRAM exactly once")
        roof["frac_of_8tbs"] = achieved / HBM_SPEC_GBS
    spec_t = sum(roofline_seconds(j["cost"], HBM_SPEC_GBS, DENSE_SPEC_TFLOPS, SPARSE_SPEC_TFLOPS)[0] for j in jobs)
    meas_t = sum(roofline_seconds(j["cost"], peaks["hbm_gbs"], peaks["bf16_tflops_sustained"],
                                  2 * peaks["bf16_tflops_sustained"])[0] for j in jobs)

    # ---- end to end through the host-buffer entry point (H2D of X and D2H of Y inside the timed region)
    # one pinned arena for all X and one for all Y, staged in device arenas in the same order: the entry point
    # then merges the step's copies into one transfer each way (the bytes copied are the same)
    nx, ny = sum(j["X"].numel() for j in jobs), sum(j["Y"].numel() for j in jobs)
    xh_arena, yh_arena = torch.empty(nx, dtype=torch.bfloat16).pin_memory(), torch.empty(ny, dtype=torch.bfloat16).pin_memory()
    xd_arena, yd_arena = torch.empty(nx, dtype=torch.bfloat16, device=dev), torch.empty(ny, dtype=torch.bfloat16, device=dev)
    ejobs, ox, oy = [], 0, 0
    for j in jobs:
        sx, sy = j["X"].numel(), j["Y"].numel()
        e = dict(j, Xh=xh_arena[ox:ox + sx].view(j["X"].shape), Yh=yh_arena[oy:oy + sy].view(j["Y"].shape),
                 X=xd_arena[ox:ox + sx].view(j["X"].shape), Y=yd_arena[oy:oy + sy].view(j["Y"].shape))
        e["Xh"].copy_(j["X"].cpu())
        ejobs.append(e)
        ox, oy = ox + sx, oy + sy
    e2e_steps = max(3, min(args.steps, 200))

    host_batch = B.make_host_batch(ejobs)    # the step as one C-ABI call: copies in, GEMMs, copies out, one sync

    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    e2e_chunks = args.e2e_chunks or (2 if (nx + ny) * 2 < 32e6 else 8)

    def e2e_step():
        # copies in, GEMMs and copies out of consecutive quarters of the step overlap on three streams
        B.patch_gemm_host_batch_pipelined(host_batch, s_in, s_out, n_chunks=e2e_chunks, weights_static=True)
    for _ in range(3):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = replicas.max_over_ranks(e2e_s, dev)
    h2d = sum(j["X"].numel() * 2 for j in jobs)
    d2h = sum(j["Y"].numel() * 2 for j in jobs)

    # ---- per-case table (each GEMM on rotating copies of its packed weight so reads come from HBM)
    table = per_case_table(torch, B, jobs, args.launch, peaks, args.variant) if args.detail and rank == 0 else []

    # ---- parity of what the timed graph computed (opt-in), and the tensor-core half of the metric
    parity = None
    if args.check != "none" and rank == 0 and world == 1 and not args.workload.startswith("stack"):
        step_graph.replay()
        torch.cuda.synchronize()
        parity = parity_check(torch, jobs)
    prefill = None
    if args.workload == "decode" and not args.no_prefill and rank == 0:
        del step_graph, multi_graph
        prefill = prefill_section(args, torch, B, dev, peaks)

    if rank != 0:
        return
    cpu, _ = oracle_sample(cases, args.cpu_budget) if world == 1 else (None, 0)
    out = {
        "metric": "hybrid_tile_gemm_effective_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_label(args),
                   "gemms_per_step": len(jobs), "tile": "128x128",
                   "packed_weight_bytes": weight_bytes,
                   "l2": "inputs larger than L2: each step streams all packed matrices once per M",
                   "multi_gpu": "replicas only" if world > 1 else "single gpu", "cuda_graph": True,
                   "steps_per_graph": spg,
                   "launch": args.launch,
                   "launch_promises": ("weights, input and output static: no launch between two drains of the GPU reads "
                                       "another's output or writes another's output buffer") if args.launch == "independent"
                                      else "weights static"},
        "us_per_gemm": step_s / len(jobs) * 1e6,
        "frac_of_roofline_spec": spec_t / step_s, "frac_of_roofline_measured": meas_t / step_s,
        "roofline": roof,
        "e2e": {"value": world * step_flops / e2e_s / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3},
        other + "_launch": {"value": world * step_flops / other_s / 1e12, "unit": "TFLOP/s",
                            "ms_per_step": other_s * 1e3, "frac_of_roofline_measured": meas_t / other_s},
        "one_step_per_graph": {"value": world * step_flops / single_s / 1e12, "unit": "TFLOP/s", "ms_per_step": single_s * 1e3,
                               "frac_of_roofline_spec": spec_t / single_s, "frac_of_roofline_measured": meas_t / single_s},
        "replay_stats": replay_stats,
        "gpu_launches": args.steps * len(jobs),
        "clocks": clocks,
        # whole calls, one per matrix, read + written bytes: patch_pack_dev (flags on the device, one kernel) and
        # patch_pack (flags on the host: table built on the host and copied from pageable memory, one kernel)
        "pack": {"gbs": pack_bytes / pack_dev_secs / 1e9, "frac_of_measured_hbm": pack_bytes / pack_dev_secs / 1e9 / peaks["hbm_gbs"],
                 "entry": "patch_pack_dev",
                 "host_flags_entry_gbs": pack_bytes / pack_secs / 1e9},
    }
    if cpu is not None:
        out["cpu_baseline"] = cpu
    if table:
        out["cases"] = table
        sp = speedup_table(table)
        if sp:
            out["speedup_vs_all_dense"] = sp
    if parity is not None:
        out["parity"] = parity
    if prefill is not None:
        out["prefill"] = prefill
    print(json.dumps(out))


# ---------------------------------------------------------------------------------------------
# block workload: the linear layers of a decoder stack chained the way a decoder chains them


def run_block(args):
    """`--workload block`: 32 LLaMA-2-7B-shaped blocks, four launches per block, M tokens (`--stack-m`):
      qkv   one stacked weight (N = 12288), X = the block's input buffer, which no GEMM writes: both promises;
      o     X = the v slice of what the qkv launch just wrote (row pitch 12288): weights promise only;
      mlp   silu(gate) * up from one stacked, interleaved gate/up weight (patch_gemm_gated), X = o's output: weights promise;
      down  X = the gated product: weights promise only.
    Three of the four launches of a block read what the launch before them wrote, as in a decoder (what sits between
    them there -- attention, norms, residuals -- is not part of this path).  Per-matrix 2:4-tile fractions ~ U[0, 1] as in
    the stack workloads; weights drawn on the device.  Reported beside it: the same launches all declared independent
    (what the stack workloads time; not a valid promise here) and all without any promise."""
    import torch
    from paper_2509_23410_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("the block workload is a single-GPU measurement")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B.lib()
    peaks = measured_peaks()
    M = args.stack_m
    cases = inputs.stack_fused_cases()
    gen = torch.Generator(device=dev)
    h = torch.empty((M, 4096), dtype=torch.bfloat16, device=dev).normal_(0.0, 1.0, generator=gen)
    launches, nbytes, flops, weight_bytes = [], 0.0, 0.0, 0
    ws = None
    for i, c in enumerate(cases):
        gen.manual_seed(inputs.MASTER_SEED * 1000 + i)
        W = torch.empty((c["N"], c["K"]), dtype=torch.bfloat16, device=dev).normal_(0.0, 0.02, generator=gen)
        flags = inputs.case_flags(c)
        role = c["name"].rsplit(".", 1)[1]
        if role == "gate_up":
            half = c["N"] // 2
            W = B.interleave_row_blocks(W[:half], W[half:]).contiguous()
            flags = B.interleave_row_blocks(flags[:half // 128], flags[half // 128:], block=1)
        layout = B.patch_packed_size(c["N"], c["K"], flags)
        packed = torch.empty(layout.total_bytes, dtype=torch.uint8, device=dev)
        B.patch_pack(W, flags, layout=layout, out=packed)
        del W
        n_out = c["N"] // 2 if role == "gate_up" else c["N"]
        Y = torch.empty((M, n_out), dtype=torch.bfloat16, device=dev)
        if role == "qkv":
            X = h
        elif role == "o":
            X = launches[-1]["Y"][:, 8192:12288]          # the v slice of the stacked qkv output
        else:
            X = launches[-1]["Y"]
        if ws is None:
            ws = torch.zeros(max(B.patch_gemm_workspace_size(layout, M), 256), dtype=torch.uint8, device=dev)
        gws = None
        if role == "gate_up":
            gws = torch.zeros(max(B.patch_gemm_gated_workspace_size(layout, M), 256), dtype=torch.uint8, device=dev)
        launches.append(dict(role=role, layout=layout, packed=packed, X=X, Y=Y, gws=gws))
        T = (c["N"] // 128) * (c["K"] // 128)
        nbytes += layout.payload_bytes + 16 * T + M * c["K"] * 2 + M * n_out * 2
        flops += 2.0 * M * 16384 * T
        weight_bytes += layout.total_bytes

    def enqueue(mode):
        for L in launches:
            if mode == "faithful":
                fl = B.WEIGHTS_STATIC | (B.INPUT_STATIC if L["role"] == "qkv" else 0)
            else:
                fl = {"independent": B.WEIGHTS_STATIC | B.INPUT_STATIC, "no-promise": 0}[mode]
            if L["role"] == "gate_up":
                B.patch_gemm_gated(L["X"], L["layout"], L["packed"], Y=L["Y"], workspace=L["gws"], flags=fl)
            else:
                B.patch_gemm(L["X"], L["layout"], L["packed"], Y=L["Y"], workspace=ws, variant=fl)

    def graph_of(mode):
        enqueue(mode)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            enqueue(mode)
        return g

    steps, warm = max(3, min(args.steps, 200)), max(args.warmup, 3)
    g = graph_of("faithful")
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    sampler.start()
    for _ in range(warm):
        g.replay()
    torch.cuda.synchronize()
    t0 = time.time()
    step_s = time_graph(torch, g, steps)
    clocks = sampler.stop(t0, time.time())
    others = {}
    for mode in ("independent", "no-promise"):
        go = graph_of(mode)
        for _ in range(3):
            go.replay()
        others[mode] = time_graph(torch, go, max(3, steps // 4))
        del go
    roof_spec = nbytes / (HBM_SPEC_GBS * 1e9) if M <= 64 else None
    out = {
        "metric": "hybrid_tile_gemm_effective_tflops", "value": flops / step_s / 1e12, "unit": "TFLOP/s", "n_gpus": 1,
        "steps": steps, "warmup": warm, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (weights drawn on the device)",
        "config": {"workload": f"llama2-7b decoder-block chain of linears (qkv -> o -> silu(gate)*up -> down, 32 blocks), M={M}",
                   "launches_per_step": len(launches), "packed_weight_bytes": weight_bytes, "cuda_graph": True,
                   "l2": "inputs larger than L2: a step streams every packed matrix once",
                   "launch": "qkv with both promises; o, mlp and down with the weights promise only (each reads what the launch before it wrote)"},
        "gbs": nbytes / step_s / 1e9,
        "frac_of_roofline_spec": (roof_spec / step_s) if roof_spec else None,
        "frac_of_roofline_measured": (nbytes / (peaks["hbm_gbs"] * 1e9) / step_s) if M <= 64 else None,
        "all_declared_independent": {"ms_per_step": others["independent"] * 1e3,
                                     "note": "what the stack workloads time; not a valid promise for this chain"},
        "no_promise": {"ms_per_step": others["no-promise"] * 1e3},
        "gpu_launches": steps * len(launches),
        "clocks": clocks,
    }
    print(json.dumps(out))


# ---------------------------------------------------------------------------------------------
# mask-learning workload: one training-forward evaluation of the soft masks of one transformer block


MASK_BYTES_PER_ELEMENT = 10.0      # soft mask: 2 B of W + 6 B of 2:4 logits read, 2 B of masked weight written
# warp instructions per group of four weights per lane of soft_mask_kernel<noise>, and its DRAM traffic per
# algorithmic byte, from the ncu capture summarised in profiles/soft_mask_kernel_llama7b_block.md
# (32 287 744 instructions for a 4096 x 4096 launch; 152.3 MB read + written against 167.8 MB)
MASK_WARP_INST_PER_GROUP = 246.3
MASK_TRAFFIC_RATIO = 0.91


def run_masks(args):
    """`--workload masks`: a step = patch_soft_mask (Gumbel noise on) over the seven linear weights of one
    LLaMA-2-7B-shaped block (4 x 4096^2, 2 x 11008x4096, 4096x11008; 1.2 GB of logits per step, so every
    byte comes from HBM).  Also times the no-noise variant, patch_hard_mask and patch_pack_patterns."""
    import torch
    from paper_2509_23410_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("the masks workload is a single-GPU measurement")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B.lib()
    peaks = measured_peaks()
    tau, kappa = 0.5, 120.0           # mid-schedule values between (2, 25) and (0.05, 350)
    shapes = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    mats = []
    for i, (N, K) in enumerate(shapes):
        W = torch.from_numpy(np.ascontiguousarray(inputs.weight(N, K, inputs.MASTER_SEED, "masks", i)).view(np.int16)).to(dev).view(torch.bfloat16)
        PT = torch.from_numpy(inputs.tile_logits(N // 128, K // 128, 0.5, inputs.MASTER_SEED, "masks", i)).to(dev)
        P6 = torch.from_numpy(inputs.pattern_logits(N, K, inputs.MASTER_SEED, "masks", i)).to(dev)
        Gw = torch.from_numpy(np.ascontiguousarray(inputs.normal_bf16((N, K), 1.0, inputs.MASTER_SEED, "masks-gw", i)).view(np.int16)).to(dev).view(torch.bfloat16)
        mats.append(dict(N=N, K=K, W=W, PT=PT, P6=P6, Wt=torch.empty_like(W), Gw=Gw, gPT=torch.empty_like(PT), gP6=torch.empty_like(P6),
                         sums=torch.empty(4, dtype=torch.float64, device=dev),
                         ws=torch.empty(B.patch_soft_mask_workspace_size(N, K), dtype=torch.uint8, device=dev),
                         flags=torch.empty((N // 128) * (K // 128), dtype=torch.uint8, device=dev),
                         patterns=torch.empty(N * K // 4, dtype=torch.uint8, device=dev)))
    elements = sum(m["N"] * m["K"] for m in mats)

    def soft(flags):
        for i, m in enumerate(mats):
            B.patch_soft_mask(m["W"], m["PT"], m["P6"], tau, kappa, 1000 + i, flags, Wt=m["Wt"], sums=m["sums"],
                              workspace=m["ws"])

    def backward():
        for i, m in enumerate(mats):
            B.patch_soft_mask_backward(m["W"], m["PT"], m["P6"], tau, kappa, m["Gw"], 1e-9, 1e-3, seed=1000 + i,
                                       gP_tile=m["gPT"], gP24=m["gP6"])

    def hard():
        for m in mats:
            B.patch_hard_mask(m["PT"], m["P6"], m["N"], m["K"], flags_out=m["flags"], patterns_out=m["patterns"])

    def graph_of(fn):
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            fn()
        torch.cuda.current_stream().wait_stream(s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    def time_graph(g, reps, warm=3):
        for _ in range(warm):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / reps

    steps = min(args.steps, 200)
    g_noise = graph_of(lambda: soft(0))
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    sampler.start()
    t0 = time.time()
    step_s = time_graph(g_noise, steps, max(args.warmup, 3))
    clocks = sampler.stop(t0, time.time())
    t_plain = time_graph(graph_of(lambda: soft(B.MASK_NO_NOISE)), 50)
    t_hard = time_graph(graph_of(hard), 50)
    t_bwd = time_graph(graph_of(backward), 50)
    # packing with the hard masks just computed (the flags visit the host only to size the buffers)
    hard()
    torch.cuda.synchronize()
    pk = []
    for m in mats:
        fl = m["flags"].cpu().numpy()
        L = B.patch_packed_size(m["N"], m["K"], fl)
        pk.append((m, fl, L, torch.empty(L.total_bytes, dtype=torch.uint8, device=dev)))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_pack, pack_bytes = 0.0, 0.0
    for rep in range(4):
        torch.cuda.synchronize()
        e0.record()
        for m, fl, L, out in pk:
            B.patch_pack_dev(m["W"], m["flags"], patterns=m["patterns"], out=out)
        e1.record()
        torch.cuda.synchronize()
        if rep:
            t_pack += e0.elapsed_time(e1) * 1e-3 / 3
    pack_bytes = sum(m["N"] * m["K"] * 2.25 + L.total_bytes for m, fl, L, out in pk)
    # end to end: logits and weights from pinned host memory every step, the four sums per matrix read back
    host = [dict(W=m["W"].cpu().pin_memory(), PT=m["PT"].cpu().pin_memory(), P6=m["P6"].cpu().pin_memory(),
                 sums=torch.empty(4, dtype=torch.float64).pin_memory()) for m in mats]
    def e2e_step():
        for m, h in zip(mats, host):
            m["W"].copy_(h["W"], non_blocking=True)
            m["PT"].copy_(h["PT"], non_blocking=True)
            m["P6"].copy_(h["P6"], non_blocking=True)
        soft(0)
        for m, h in zip(mats, host):
            h["sums"].copy_(m["sums"], non_blocking=True)
        torch.cuda.synchronize()
    e2e_step()
    tw = time.time()
    for _ in range(3):
        e2e_step()
    e2e_s = (time.time() - tw) / 3
    h2d = sum(h["W"].numel() * 2 + h["PT"].numel() * 4 + h["P6"].numel() * 4 for h in host)
    reg = B.patch_mask_regularizers(np.stack([h["sums"].numpy() for h in host]), 0.75, 7.0, 10.0)
    # the oracle on a bounded sample: one 1024 x 1024 matrix with noise
    import oracle
    Wc, PTc, P6c = inputs.weight(1024, 1024, 1, "masks-cpu"), inputs.tile_logits(8, 8, 0.5, 1, "masks-cpu"), \
        inputs.pattern_logits(1024, 1024, 1, "masks-cpu")
    tc = time.time()
    oracle.soft_mask(Wc, PTc, P6c, tau, kappa, seed=1, noise=True)
    tc = time.time() - tc
    gbs = elements * MASK_BYTES_PER_ELEMENT / step_s / 1e9
    winst = MASK_WARP_INST_PER_GROUP * elements / 4 / 32           # warp instructions per step
    alu_peak = 148 * 4 * (clocks.get("sm_mhz") or 1965.0) * 1e6    # warp instructions per second
    out = {
        "metric": "soft_mask_forward_effective_gbs", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "soft-mask forward (Eq. 2-5) of one llama2-7b block's seven linear weights, Gumbel noise on",
                   "tau": tau, "kappa": kappa, "elements": elements, "cuda_graph": True,
                   "l2": "inputs larger than L2: 2.0 GB streamed per step"},
        # with the noise on the kernel is bound by instruction issue (integer mixes, two logarithms and one
        # exponential per candidate): achieved = warp instructions per second, peak = 148 SMs x 4 schedulers x
        # one warp instruction per clock at the SM clock sampled during the run
        "roofline": {"bound": "alu", "achieved": winst / step_s / 1e9, "peak": alu_peak / 1e9, "unit": "Gwarp-inst/s",
                     "frac": winst / step_s / alu_peak,
                     "traffic": MASK_TRAFFIC_RATIO * elements * MASK_BYTES_PER_ELEMENT / len(mats),
                     "kernel": "soft_mask_kernel<noise>", "hbm_gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                     "peak_source": "148 x 4 x sampled SM clock; instructions per group from ncu"},
        "soft_mask_no_noise": {"ms_per_step": t_plain * 1e3, "gbs": elements * MASK_BYTES_PER_ELEMENT / t_plain / 1e9,
                               "frac_of_measured_hbm": elements * MASK_BYTES_PER_ELEMENT / t_plain / 1e9 / peaks["hbm_gbs"]},
        "hard_mask": {"ms_per_step": t_hard * 1e3, "gbs": elements * 6.25 / t_hard / 1e9,
                      "frac_of_measured_hbm": elements * 6.25 / t_hard / 1e9 / peaks["hbm_gbs"]},
        "soft_mask_backward": {"ms_per_step": t_bwd * 1e3, "gbs": elements * 16.0 / t_bwd / 1e9,
                               "frac_of_measured_hbm": elements * 16.0 / t_bwd / 1e9 / peaks["hbm_gbs"],
                               "note": "16 B per element: W, Gw and six logits read, six logit gradients written; noise on"},
        "pack_patterns": {"ms_per_step": t_pack * 1e3, "gbs": pack_bytes / t_pack / 1e9,
                          "note": "patch_pack_dev with the flags and candidates patch_hard_mask left on the device"},
        "e2e": {"value": elements * MASK_BYTES_PER_ELEMENT / e2e_s / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": 32 * len(mats), "ms_per_step": e2e_s * 1e3},
        "regularizers_of_last_step": reg,
        "gpu_launches": steps * 2 * len(mats),
        "clocks": clocks,
        "cpu_baseline": {"value": 1024 * 1024 * MASK_BYTES_PER_ELEMENT / tc / 1e9, "unit": "GB/s", "cores": 1,
                         "kind": "oracle", "sample": "one 1024x1024 matrix, noise on"},
    }
    print(json.dumps(out))


def workload_label(args):
    return {"13b": "llama2-13b linears", "stack": f"llama2-7b full linear stack, M={args.stack_m}",
            "stack-fused": f"llama2-7b full linear stack with q/k/v and gate/up stacked, M={args.stack_m}",
            "single": "single 1024x1024 GEMM",
            "decode-q4": "llama2-7b decode linears, every tile stored with 4-bit values"}.get(args.workload, f"llama2-7b {args.workload} linears")


def B_kernel_name(M, launch="independent"):
    if M <= 64:
        return "decode_cluster_kernel" if launch == "independent" else "decode_kernel"
    return "prefill2_kernel (two row-blocks per CTA) or prefill_kernel, chosen per shape"


# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes per launch, from the ncu captures
# summarised in profiles/decode_cluster_kernel_llama7b_decode.md (1.055, 1.018, 1.007) and
# profiles/decode_kernel_llama7b_decode.md (1.035, 1.029, 1.008).
# Traffic grows in proportion to the payload, so the ratio scales to any launch of the kernel.
# profiles/decode_q4_kernel_llama7b_decode_q4.md: 1.006, 1.006, 1.007 (reads only; nothing is written to DRAM).
NCU_TRAFFIC_RATIO = {"decode_kernel": 1.03, "decode_cluster_kernel": 1.03, "decode_q4_kernel": 1.006}


def load_traffic(kernel, algorithmic):
    r = NCU_TRAFFIC_RATIO.get(kernel)
    return None if r is None else r * algorithmic


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="decode", choices=["decode", "prefill", "13b", "single", "stack", "stack-fused", "block", "masks", "decode-q4"])
    ap.add_argument("--stack-m", type=int, default=1, help="tokens per GEMM of the 224-GEMM stack workload")
    ap.add_argument("--launch", default="independent", choices=["dependent", "independent"],
                    help="independent (default; true for this workload, whose GEMMs do not feed each other): "
                         "the caller promises X is not produced by the preceding kernel; dependent: every "
                         "GEMM waits for the previous one before reading X")
    ap.add_argument("--variant", type=int, default=0, help="0 auto, 1 decode GEMV (M <= 4), 2 tensor-core kernel")
    ap.add_argument("--detail", action="store_true", help="add the per-GEMM table (us, TFLOP/s, roofline fraction)")
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--steps-per-graph", type=int, default=8,
                    help="consecutive steps captured into one CUDA graph (the timed region still runs exactly --steps steps)")
    ap.add_argument("--check", default="none", choices=["none", "sampled"],
                    help="sampled: after timing, compare the outputs of the timed graph with the CPU oracle and print "
                         "parity {relF, maxrel} on the line (adds the oracle's run time)")
    ap.add_argument("--no-prefill", action="store_true",
                    help="default workload only: skip the prefill section (the tensor-core half of the metric)")
    ap.add_argument("--e2e-chunks", type=int, default=0,
                    help="runs of jobs the end-to-end leg pipelines over its three streams (0: 2 for steps that move "
                         "less than 32 MB, where each extra run costs more in event traffic than it hides, else 8)")
    args = ap.parse_args()
    if args.workload == "masks":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the masks workload reports the oracle in its cpu_baseline key"}))
        else:
            run_masks(args)
    elif args.workload == "block":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the block workload has no oracle arm; see the decode workload"}))
        else:
            run_block(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
