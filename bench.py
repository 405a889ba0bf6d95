#!/usr/bin/env python
"""Benchmark of the adapted quantized linear layer (Q-BLoRA / QA-BLoRA hot path) on B200.

One step = forward + backward (dX, dA, dB) of every adapted linear of the workload through the
C-ABI library, inputs resident in HBM.  The headline workload is the largest single-GPU configuration
(the 13B-shaped decoder layer of seven linears); the other fine-tuning configurations are timed after it and
reported under ``configs``.  A timed region is exactly ``--steps`` steps; it is repeated until about 1.5 s of
timed work have run, so the clocks sampled beside it are those of a sustained run.  Prints ONE JSON line.
``--impl reference`` times the fp64 CPU oracle on the host cores instead (a bounded sample of the same
workload per step).

Multi-GPU: the path has no exchange step; ``--gpus N`` (launched with torch.distributed.run) runs
N independent replicas and reports the aggregate ("replicas only", weak scaling).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2407_17029_b200 import synth  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel come from profiles/dram_traffic.json, which
# records, next to each figure, the SHA-256 of the kernel source it was captured on: a figure whose kernel has
# changed since is reported as null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")
DOMINANT_KERNEL_SOURCE = os.path.join(ROOT, "paper_2407_17029_b200", "csrc", "tc_gemm.cu")
BURST_REGION_S = 0.1    # a timed region shorter than this runs at boost clocks: compare with the burst peak


def measured_traffic(workload, geometry):
    """(bytes per launch, note) of the dominant kernel from the ncu capture on record, or (None, why)."""
    try:
        import hashlib
        rec = json.load(open(TRAFFIC_FILE))
        sha = hashlib.sha256(open(DOMINANT_KERNEL_SOURCE, "rb").read()).hexdigest()
        for e in rec["entries"]:
            if e["workload"] == workload and e["geometry"] == geometry:
                if e["kernel_source_sha256"] != sha:
                    return None, "kernel source changed since the ncu capture on record"
                return float(e["dram_bytes_per_launch"]), e.get("note", "ncu capture, profiles/")
        return None, "no ncu capture on record for this workload"
    except Exception as ex:   # missing file: no figure
        return None, f"no traffic record ({type(ex).__name__})"


METRIC = "fused 4-bit+BLoRA linear fwd+bwd TFLOP/s & low-bit GEMM GB/s, % of roofline"


# ----------------------------------------------------------------------------------- accounting
SCALE_OP = 0   # adapter operator pair of the run (--scale-op)


def linear_flops(T, d_out, d_in, r, geom):
    """Algorithmic flops of one adapted linear, forward + backward: two base contractions
    (2*T*D_in*D_out each) and the adapter's (2*T*r*(P+Q) forward, twice that backward)."""
    P, Q = d_in // geom.lambda_in, d_out // geom.lambda_out
    base = 2 * (2.0 * T * d_in * d_out)
    adapter = 3 * (2.0 * T * r * (P + Q))
    return base, adapter


def packed_bytes(d_out, d_in, block_in=64, with_beta=True):
    """Algorithmic bytes of one pass over a packed weight: 4-bit codes + fp32 alpha (+ beta) per block."""
    return d_out * d_in // 2 + (d_out * d_in // block_in) * (8 if with_beta else 4)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ reference (oracle)
def oracle_step(wl, geom, sample_rows, cache):
    """One bounded oracle step: forward + backward of every linear on `sample_rows` token rows."""
    import oracle
    flops = 0.0
    t0 = time.perf_counter()
    for spec in wl.linears:
        qw, Wt, li = cache[spec.name]
        ad = oracle.Adapter(geom.lambda_in, geom.lambda_out, wl.rank, wl.scaling, li.A, li.B, SCALE_OP)
        oracle.linear_fwd(Wt, ad, li.X)
        oracle.linear_bwd(Wt, ad, li.X, li.dY)
        b, a = linear_flops(sample_rows, spec.d_out, spec.d_in, wl.rank, geom)
        flops += b + a
    return time.perf_counter() - t0, flops


def oracle_cache(wl, geom, sample_rows):
    import oracle
    cache = {}
    for spec in wl.linears:
        li = synth.make_linear_inputs(wl, spec, geom, seed=0, tokens=sample_rows)
        qw = oracle.quantize_blockwise(li.W, wl.block_in, 1, wl.qfmt)
        cache[spec.name] = (qw, oracle.dequantize(qw), li)
        li.W = None
    return cache


def run_reference(args, wl, geom):
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = ref_rows_for(wl, geom, args.ref_rows)
    cache = oracle_cache(wl, geom, rows)
    for _ in range(min(args.warmup, 1)):
        oracle_step(wl, geom, rows, cache)
    tot_t, tot_f = 0.0, 0.0
    steps = min(args.steps, args.ref_max_steps)
    for _ in range(steps):
        t, f = oracle_step(wl, geom, rows, cache)
        tot_t += t; tot_f += f
    val = tot_f / tot_t / 1e12
    cores = oracle.num_threads()
    sample = f"{rows} of {wl.tokens} token rows per step, all linears, fwd+bwd (dX, dA, dB)"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": tot_t / steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": wl.name, "geometry": geom.name, "scale_op": SCALE_OP, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------- GPU arm
class GpuCtx:
    """Device, rank and process-group plumbing shared by the measurements of one run."""

    def __init__(self):
        import torch
        from paper_2407_17029_b200 import binding as qb
        self.torch, self.qb = torch, qb
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=self.dev)
            self.dist = dist
        self.peaks = measured_peaks()
        self.l2_bytes = torch.cuda.get_device_properties(self.dev).L2_cache_size

    def bf(self, a):
        return self.torch.from_numpy(synth.bf16_bits(a).view(np.int16).copy()).to(self.dev).view(self.torch.bfloat16)

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, x):
        if self.dist is None:
            return float(x)
        t = self.torch.tensor([x], dtype=self.torch.float64, device=self.dev)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())


def measure_workload(ctx, wl, geom, steps, warmup, min_region_s, no_graph=False, want_e2e=True):
    """Times forward + backward steps of one workload.  A timed region is EXACTLY `steps` steps between a barrier +
    synchronize on both sides; the region is repeated until at least `min_region_s` seconds of timed work have
    run (so that clocks and power settle where a long job would hold them), and the mean region is reported."""
    torch, qb, dev = ctx.torch, ctx.qb, ctx.dev
    T, r = wl.tokens, wl.rank
    # ---- resident buffers; rotate over enough distinct sets to exceed 2x L2
    lin = []
    step_bytes = 0
    for spec in wl.linears:
        li = synth.make_linear_inputs(wl, spec, geom, seed=ctx.rank)
        dq = qb.quantize_blockwise(torch.from_numpy(li.W).to(dev), wl.block_in, 1, wl.qfmt)
        li.W = None
        step_bytes += (li.X.size + li.dY.size) * 2 * 2 + packed_bytes(spec.d_out, spec.d_in, wl.block_in, wl.qfmt == 1)
        lin.append((spec, li, dq))
    nsets = max(2, int(np.ceil(2.0 * ctx.l2_bytes / step_bytes)) + 1)
    sets = []
    for s in range(nsets):
        items = []
        for spec, li, dq in lin:
            # distinct device copies (same values): what matters is that the addresses differ
            q2 = qb.QWeight(dq.d_out, dq.d_in, dq.block_in, dq.block_out, dq.qfmt, dq.code,
                            dq.codes.clone(), dq.alpha.clone(), dq.beta.clone() if dq.beta is not None else None)
            ad = qb.Adapter(geom.lambda_in, geom.lambda_out, r, wl.scaling, ctx.bf(li.A), ctx.bf(li.B), SCALE_OP)
            X, dY = ctx.bf(li.X), ctx.bf(li.dY)
            Y = torch.empty((T, spec.d_out), dtype=torch.bfloat16, device=dev)
            dX = torch.empty((T, spec.d_in), dtype=torch.bfloat16, device=dev)
            dA = torch.empty(tuple(ad.A.shape), dtype=torch.float32, device=dev)
            dB = torch.empty(tuple(ad.B.shape), dtype=torch.float32, device=dev)
            wsf = qb.alloc_workspace(qb.OP_LINEAR_FWD, q2, ad, T)
            wsb = qb.alloc_workspace(qb.OP_LINEAR_BWD, q2, ad, T)
            items.append((spec, q2, ad, X, dY, Y, dX, dA, dB, wsf, wsb))
        sets.append(items)
    del lin

    def step(i, ev=None):
        for j, (spec, q2, ad, X, dY, Y, dX, dA, dB, wsf, wsb) in enumerate(sets[i % nsets]):
            if ev is not None and j == ev[2]:
                qb.set_timing_events(ev[0], ev[1])
            qb.linear_fwd(q2, ad, X, ws=wsf, out=Y)
            qb.linear_bwd(q2, ad, X, dY, ws=wsb, outs=(dX, dA, dB))

    flops_step = sum(sum(linear_flops(T, s.d_out, s.d_in, r, geom)) for s in wl.linears)
    # dominant kernel: the forward base contraction of the largest linear
    dom = max(range(len(wl.linears)), key=lambda j: wl.linears[j].d_out * wl.linears[j].d_in)
    dspec = wl.linears[dom]
    dom_flops = 2.0 * T * dspec.d_in * dspec.d_out

    for i in range(warmup):
        step(i)
    ctx.barrier()
    graphs = None
    if not no_graph:
        # the same steps as CUDA graphs (one graph per buffer set, one step each): the small adapter-side kernels
        # are launch-bound when issued from the host one by one
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graphs = []
        for si in range(nsets):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                step(si)
            graphs.append(g)
        for i in range(warmup):
            graphs[i % nsets].replay()
        ctx.barrier()

    def run_steps(first):
        for i in range(steps):
            if graphs is not None:
                graphs[(first + i) % nsets].replay()
            else:
                step(first + i)

    sampler = ClockSampler(ctx.local)
    sampler.start()
    time.sleep(0.25)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    regions = []
    done_s, k = 0.0, 0
    while not regions or (done_s < min_region_s and len(regions) < 2000):
        ctx.barrier()
        e0.record()
        run_steps(warmup + k * steps)
        e1.record()
        ctx.barrier()
        regions.append(e0.elapsed_time(e1))
        done_s += regions[-1] * 1e-3
        k += 1
    # ---- one more region with every call launched from the host; the library brackets the dominant kernel of
    # each step with an event pair (the chip is in the state the regions above left it in)
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), dom) for _ in range(steps)]
    for a, b, _ in kev:          # torch creates the CUDA event handle on first record
        a.record(); b.record()
    launches0 = qb.kernel_launches()
    ctx.barrier()
    e0.record()
    for i in range(steps):
        step(warmup + i, kev[i])
    e1.record()
    ctx.barrier()
    launches = qb.kernel_launches() - launches0
    eager_ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    dom_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in kev)
    if graphs is None:
        regions.append(eager_ms)
    for spec, q2, ad, X, dY, Y, dX, dA, dB, wsf, wsb in sets[0]:
        assert qb.device_status(wsf) == qb.OK and qb.device_status(wsb) == qb.OK
    ms = ctx.max_over_ranks(statistics.mean(regions))          # mean region of exactly `steps` steps, max over ranks
    value = flops_step * ctx.world * steps / (ms * 1e-3) / 1e12
    timed_s = sum(regions) * 1e-3 + eager_ms * 1e-3
    sustained = timed_s >= BURST_REGION_S
    peak = ctx.peaks["bf16_tflops_sustained"] if sustained else ctx.peaks["bf16_tflops"]
    achieved = dom_flops / (dom_ms * 1e-3) / 1e12
    traffic, traffic_note = measured_traffic(wl.name, geom.name)
    res = {
        "value": value, "ms_per_step": ms / steps, "steps": steps, "regions": len(regions),
        "region_ms": {"mean": statistics.mean(regions), "min": min(regions), "max": max(regions)},
        "timed_s": timed_s, "step_flops": flops_step, "clocks": clocks, "gpu_launches": int(launches),
        "launch": "eager launches" if graphs is None else "CUDA-graph replay, one graph per buffer set",
        "l2": f"rotating over {nsets} distinct buffer sets ({nsets * step_bytes / 2**20:.0f} MiB > 2x L2)",
        "frac_of_peak": value / ctx.world / peak,
        "roofline": {"bound": "tensor", "kernel": f"forward base contraction {dspec.name}[{dspec.d_out},{dspec.d_in}] T={T}",
                     "achieved": achieved, "peak": peak,
                     "peak_kind": (f"bf16 dense, {'sustained' if sustained else 'burst'}, {ctx.peaks['source']}: the kernel was timed inside "
                                   f"{timed_s:.2f} s of back-to-back steps (burst figure below {BURST_REGION_S} s, sustained above)"),
                     "unit": "TFLOP/s", "frac": achieved / peak,
                     "frac_of_burst": achieved / ctx.peaks["bf16_tflops"], "frac_of_sustained": achieved / ctx.peaks["bf16_tflops_sustained"],
                     "traffic": traffic, "traffic_note": traffic_note, "ms_per_launch": dom_ms},
        "eager": {"ms_per_step": eager_ms / steps, "value": flops_step * steps / (eager_ms * 1e-3) / 1e12,
                  "unit": "TFLOP/s", "note": "this rank, every call launched from the host"}}
    if not want_e2e:
        return res

    # ---- end to end: host (pinned) inputs in, results out, copies inside the timed region.  Three streams form
    # a pipeline over the linears of a step -- one issues the host-to-device copies, one the library calls, one
    # the device-to-host copies -- tied together per linear by events, so that the two copy directions (separate
    # copy engines, full-duplex link) and the compute overlap; the steps alternate between the device buffer sets,
    # and a buffer is written again only after its previous reader is done.  Every step still moves all of its
    # inputs and results.
    lanes = []
    h2d = d2h = 0
    lane_bytes = sum((X.numel() + dY.numel() + Y.numel() + dX.numel()) * 2 for _, _, _, X, dY, Y, dX, *_ in sets[0])
    n_lanes = max(1, min(3, nsets, int(8e9 // max(lane_bytes, 1))))        # at most ~8 GB of pinned host memory
    for li_ in range(n_lanes):
        host = []
        for spec, q2, ad, X, dY, Y, dX, dA, dB, wsf, wsb in sets[li_]:
            hX, hdY = X.cpu().pin_memory(), dY.cpu().pin_memory()
            hY, hdX = torch.empty_like(Y, device="cpu").pin_memory(), torch.empty_like(dX, device="cpu").pin_memory()
            hdA, hdB = torch.empty_like(dA, device="cpu").pin_memory(), torch.empty_like(dB, device="cpu").pin_memory()
            ev = tuple(torch.cuda.Event() for _ in range(3))                # inputs landed / calls done / results copied out
            host.append((hX, hdY, hY, hdX, hdA, hdB, ev))
            if li_ == 0:
                h2d += hX.numel() * 2 + hdY.numel() * 2
                d2h += hY.numel() * 2 + hdX.numel() * 2 + hdA.numel() * 4 + hdB.numel() * 4
        lanes.append((sets[li_], host))
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_step(i=0):
        items, host = lanes[i % n_lanes]
        for (spec, q2, ad, X, dY, Y, dX, dA, dB, wsf, wsb), (hX, hdY, hY, hdX, hdA, hdB, (ev_in, ev_run, ev_out)) in zip(items, host):
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_run)                  # the previous calls on this buffer set have read X and dY
                X.copy_(hX, non_blocking=True); dY.copy_(hdY, non_blocking=True)
                ev_in.record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in); s_run.wait_event(ev_out)   # inputs are here; the previous results are out
                qb.linear_fwd(q2, ad, X, ws=wsf, out=Y)
                qb.linear_bwd(q2, ad, X, dY, ws=wsb, outs=(dX, dA, dB))
                ev_run.record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run)
                hY.copy_(Y, non_blocking=True); hdX.copy_(dX, non_blocking=True)
                hdA.copy_(dA, non_blocking=True); hdB.copy_(dB, non_blocking=True)
                ev_out.record(s_out)

    e2e_steps = max(3, min(steps, 10))
    for i in range(n_lanes):
        e2e_step(i)
    ctx.barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(i)
    ctx.barrier()
    e2e_s = ctx.max_over_ranks(time.perf_counter() - t0)
    res["e2e"] = {"value": flops_step * ctx.world * e2e_steps / e2e_s / 1e12, "unit": "TFLOP/s",
                  "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "lanes": n_lanes,
                  "pipeline": "copy-in, compute and copy-out streams, chained per linear by events"}
    return res


def ref_rows_for(wl, geom, requested):
    """Token rows of one bounded oracle step: about 45 GF of fp64 work (10-15 s on a dozen host cores)."""
    if requested:
        return min(requested, wl.tokens)
    per_row = sum(sum(linear_flops(1, s.d_out, s.d_in, wl.rank, geom)) for s in wl.linears)
    return int(max(8, min(wl.tokens, 512, round(45e9 / per_row / 8) * 8)))


def run_gpu(args, wl, geom):
    ctx = GpuCtx()
    torch, qb = ctx.torch, ctx.qb
    m = measure_workload(ctx, wl, geom, args.steps, args.warmup, args.min_region_s, args.no_graph, want_e2e=True)
    T, r = wl.tokens, wl.rank
    line = {"metric": METRIC, "value": m["value"], "unit": "TFLOP/s", "n_gpus": ctx.world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "scale_op": SCALE_OP, "geometry": f"{geom.name} (lambda_in={geom.lambda_in}, lambda_out={geom.lambda_out})",
                       "tokens": T, "linears": [f"{s.name}[{s.d_out},{s.d_in}]" for s in wl.linears], "rank": r,
                       "quant": "4-bit, block 64 along input, " + ("min-max" if wl.qfmt else "level table + absmax"),
                       "parallelism": "replicas only" if ctx.world > 1 else "single GPU",
                       "launch": m["launch"], "l2": m["l2"],
                       "timing": f"{m['regions']} timed regions of exactly {args.steps} steps each ({m['timed_s']:.2f} s of timed work); "
                                 "value = steps x flops / mean region"},
            "regions": m["regions"], "region_ms": m["region_ms"], "frac_of_peak": m["frac_of_peak"],
            "clocks": m["clocks"], "gpu_launches": m["gpu_launches"], "e2e": m["e2e"], "roofline": m["roofline"],
            "step_flops": m["step_flops"], "eager": m["eager"]}
    # ---- the other fine-tuning configurations, each for about a second of timed work (rank 0 reports its own)
    if ctx.world == 1 and args.configs:
        line["configs"] = {}
        for name in [c for c in args.configs.split(",") if c and c != wl.name]:
            torch.cuda.empty_cache()
            w2 = synth.WORKLOADS[name]
            m2 = measure_workload(ctx, w2, geom, args.steps, args.warmup, args.min_region_s_configs, args.no_graph, want_e2e=False)
            line["configs"][name if name != "C5" else "C5 shapes as a fine-tuning step"] = {
                "tokens": w2.tokens, "linears": [f"{s.name}[{s.d_out},{s.d_in}]" for s in w2.linears],
                "ms_per_step": m2["ms_per_step"], "value": m2["value"], "unit": "TFLOP/s", "frac_of_peak": m2["frac_of_peak"],
                "regions": m2["regions"], "timed_s": m2["timed_s"], "clocks": m2["clocks"],
                "dominant_kernel": {k: m2["roofline"][k] for k in ("kernel", "achieved", "peak", "peak_kind", "frac", "frac_of_burst", "ms_per_launch")}}
    torch.cuda.empty_cache()
    if ctx.rank == 0 and not args.no_extras:
        line["lowbit"] = lowbit_extras(qb, torch, ctx.dev, ctx.peaks, ctx.l2_bytes, args.lowbit_shapes.split(","),
                                       [int(t) for t in args.lowbit_tokens.split(",")])
        torch.cuda.empty_cache()
        if not args.no_dense:
            line["dense_16bit"] = dense_extras(qb, torch, ctx.dev, ctx.peaks)
    if ctx.rank == 0 and not args.no_cpu_baseline and ctx.world == 1:
        rows = ref_rows_for(wl, geom, args.ref_rows)
        cache = oracle_cache(wl, geom, rows)
        import oracle
        t, f = oracle_step(wl, geom, rows, cache)
        line["cpu_baseline"] = {"value": f / t / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": f"{rows} of {T} token rows, all linears, fwd+bwd (dX, dA, dB), {t:.1f} s"}
    if ctx.rank == 0:
        print(json.dumps(line), flush=True)
    if ctx.dist is not None:
        ctx.dist.destroy_process_group()


def lowbit_extras(qb, torch, dev, peaks, l2_bytes, shapes=("q", "up"), tokens=(1, 16, 2048)):
    """Deploy path of the QA-BLoRA config: merge, then the low-bit product at 1 and 16 tokens on the
    attention and MLP shapes; GB/s = packed-weight bytes streamed once / kernel time."""
    wl = synth.WORKLOADS["C5"]
    out = {}

    def bf(a):
        return torch.from_numpy(synth.bf16_bits(a).view(np.int16).copy()).to(dev).view(torch.bfloat16)

    for spec in [sp for sp in wl.linears if sp.name in shapes]:
        li = synth.make_linear_inputs(wl, spec, synth.GEOM_A, seed=0, tokens=16)
        Wd = torch.from_numpy(li.W).to(dev)
        dq = qb.quantize_blockwise(Wd, 64, 1, qb.FMT_AFFINE_MINMAX)
        li.W = None
        # quantizer: reads the fp32 weight once (larger than L2), writes codes + alpha + beta
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        qb.quantize_blockwise(Wd, 64, 1, qb.FMT_AFFINE_MINMAX, out=dq)
        s.record()
        for _ in range(5):
            qb.quantize_blockwise(Wd, 64, 1, qb.FMT_AFFINE_MINMAX, out=dq)
        e.record(); torch.cuda.synchronize()
        q_us = s.elapsed_time(e) / 5 * 1e3
        q_bytes = Wd.numel() * 4 + packed_bytes(spec.d_out, spec.d_in)
        out[f"{spec.name}/quantize"] = {"us": q_us, "GB/s": q_bytes / q_us / 1e3, "frac_hbm": q_bytes / q_us / 1e3 / peaks["hbm_gbs"],
                                        "bytes": q_bytes, "note": "fp32 in (larger than L2), outputs preallocated"}
        # the same weight in the level-table format (the format of the fine-tuning configurations)
        dq0 = qb.quantize_blockwise(Wd, 64, 1, qb.FMT_CODEBOOK_ABSMAX)
        s.record()
        for _ in range(5):
            qb.quantize_blockwise(Wd, 64, 1, qb.FMT_CODEBOOK_ABSMAX, code=dq0.code, out=dq0)   # (table passed in: building the default one costs host time)
        e.record(); torch.cuda.synchronize()
        q0_us = s.elapsed_time(e) / 5 * 1e3
        q0_bytes = Wd.numel() * 4 + packed_bytes(spec.d_out, spec.d_in, with_beta=False)
        out[f"{spec.name}/quantize_level_table"] = {"us": q0_us, "GB/s": q0_bytes / q0_us / 1e3,
                                                    "frac_hbm": q0_bytes / q0_us / 1e3 / peaks["hbm_gbs"], "bytes": q0_bytes,
                                                    "note": "fp32 in (larger than L2), outputs preallocated"}
        del Wd, dq0
        ad = qb.Adapter(64, 8, wl.rank, 1.0, bf(li.A), bf(li.B))
        nbytes = packed_bytes(spec.d_out, spec.d_in)
        ncopies = int(np.ceil(2.0 * l2_bytes / nbytes)) + 1
        copies = []
        for _ in range(ncopies):
            m = qb.merge(dq, ad)
            copies.append(qb.QWeight(m.d_out, m.d_in, 64, 1, m.qfmt, m.code, m.codes.clone(), m.alpha.clone(), m.beta.clone()))
        # merge timing
        wsm = qb.alloc_workspace(qb.OP_MERGE, dq, ad, 0)
        for _ in range(3):
            qb.merge(dq, ad, ws=wsm)
        s.record()
        for _ in range(10):
            qb.merge(dq, ad, ws=wsm)
        e.record(); torch.cuda.synchronize()
        out[f"{spec.name}/merge_us"] = s.elapsed_time(e) / 10 * 1e3
        X = bf(li.X)
        for T in tokens:
            if T > 16:
                # prefill-shaped product: the fused dequant GEMM with the min-max table; tensor-bound
                Xl = bf(synth.make_activations(0, f"C5/{spec.name}/Xl", T, spec.d_in)[0])
                Yl = torch.empty((T, spec.d_out), dtype=torch.bfloat16, device=dev)
                wsl = qb.alloc_workspace(qb.OP_LOWBIT_GEMM, copies[0], None, T)
                for i in range(3):
                    qb.lowbit_gemm(copies[i % ncopies], Xl, ws=wsl, out=Yl)
                s.record()
                for i in range(10):
                    qb.lowbit_gemm(copies[i % ncopies], Xl, ws=wsl, out=Yl)
                e.record(); torch.cuda.synchronize()
                us = s.elapsed_time(e) / 10 * 1e3
                tf = 2.0 * T * spec.d_in * spec.d_out / us / 1e6
                out[f"{spec.name}/T{T}"] = {"us": us, "TFLOP/s": tf, "frac_bf16_burst": tf / peaks["bf16_tflops"],
                                            "peak_kind": "burst (ten launches, a few ms)", "frac_bf16_sustained": tf / peaks["bf16_tflops_sustained"],
                                            "status": qb.device_status(wsl)}
                del Xl, Yl
                continue
            Xt = X[:T].contiguous()
            Y = torch.empty((T, spec.d_out), dtype=torch.bfloat16, device=dev)
            ws = qb.alloc_workspace(qb.OP_LOWBIT_GEMM, copies[0], None, T)
            for i in range(5):
                qb.lowbit_gemm(copies[i % ncopies], Xt, ws=ws, out=Y)
            reps = 40
            # kernel time: an event pair recorded by the library right around the kernel of each call
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            for a, b in evs:
                a.record(); b.record()
            torch.cuda.synchronize()
            s.record()
            for i in range(reps):
                qb.set_timing_events(*evs[i])
                qb.lowbit_gemm(copies[i % ncopies], Xt, ws=ws, out=Y)
            e.record(); torch.cuda.synchronize()
            call_us = s.elapsed_time(e) / reps * 1e3
            single_us = statistics.mean(a.elapsed_time(b) for a, b in evs) * 1e3
            # chain time: >= 64 launches over the rotating copies replayed as one CUDA graph, the way a
            # decode step issues its products back to back; per-launch time = graph time / launches.  An
            # event pair around ONE launch also counts about 6 us of launch latency that a chain hides.
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            n_chain = ncopies * max(2, -(-64 // ncopies))      # >= 64 launches: a decode step issues hundreds;
                                                                # the graph's own launch cost is spread over them
            with torch.cuda.stream(side):
                qb.lowbit_gemm(copies[0], Xt, ws=ws, out=Y)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(n_chain):
                    qb.lowbit_gemm(copies[i % ncopies], Xt, ws=ws, out=Y)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            chain = []
            for _ in range(10):
                s.record(); graph.replay(); e.record(); torch.cuda.synchronize()
                chain.append(s.elapsed_time(e) / n_chain * 1e3)
            us = statistics.median(chain)
            gbs = nbytes / (us * 1e-6) / 1e9
            out[f"{spec.name}/T{T}"] = {"kernel_us": us, "timing": f"CUDA-graph chain of {n_chain} launches over {ncopies} weight copies (launches chained as programmatic dependents)",
                                        "GB/s": gbs, "frac_hbm": gbs / peaks["hbm_gbs"], "bytes": nbytes, "copies": ncopies,
                                        "single_launch_event_pair_us": single_us, "call_us_back_to_back": call_us,
                                        "status": qb.device_status(ws)}
    out["peak_hbm_gbs"] = peaks["hbm_gbs"]
    out["peak_kind"] = peaks["source"]
    return out


def dense_extras(qb, torch, dev, peaks):
    """The other deployment (Sec. 3.1 / 3.2): merge the adapter into a dense bf16 weight, then serve it with the
    library's plain bf16 tensor-core GEMM.  TFLOP/s against the burst bf16 peak (ten launches, a few ms)."""
    out = {}

    def bf(a):
        return torch.from_numpy(synth.bf16_bits(a).view(np.int16).copy()).to(dev).view(torch.bfloat16)

    for wname, lname in (("C2", "attn_proj"), ("C4", "gate")):
        wl = synth.WORKLOADS[wname]
        spec = [sp for sp in wl.linears if sp.name == lname][0]
        T = wl.tokens
        li = synth.make_linear_inputs(wl, spec, synth.GEOM_A, seed=0, tokens=T)
        dq = qb.quantize_blockwise(torch.from_numpy(li.W).to(dev), 64, 1, wl.qfmt)
        li.W = None
        ad = qb.Adapter(64, 8, wl.rank, wl.scaling, bf(li.A), bf(li.B))
        Wm = torch.empty((spec.d_out, spec.d_in), dtype=torch.bfloat16, device=dev)
        wsm = qb.alloc_workspace(qb.OP_MERGE_DENSE, dq, ad, 0)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        qb.merge_dense(dq, ad, out=Wm, ws=wsm)
        s.record()
        for _ in range(5):
            qb.merge_dense(dq, ad, out=Wm, ws=wsm)
        e.record(); torch.cuda.synchronize()
        merge_us = s.elapsed_time(e) / 5 * 1e3
        X = bf(li.X)
        Y = torch.empty((T, spec.d_out), dtype=torch.bfloat16, device=dev)
        ws = torch.empty(256, dtype=torch.uint8, device=dev)
        for _ in range(3):
            qb.dense_gemm(Wm, X, ws=ws, out=Y)
        s.record()
        for _ in range(10):
            qb.dense_gemm(Wm, X, ws=ws, out=Y)
        e.record(); torch.cuda.synchronize()
        us = s.elapsed_time(e) / 10 * 1e3
        tf = 2.0 * T * spec.d_in * spec.d_out / us / 1e6
        out[f"{wname}/{lname}[{spec.d_out},{spec.d_in}] T={T}"] = {
            "merge_dense_us": merge_us, "dense_gemm_us": us, "TFLOP/s": tf, "frac_bf16_burst": tf / peaks["bf16_tflops"],
            "peak_kind": "burst (ten launches, a few ms)", "status": qb.device_status(ws)}
        del Wm, X, Y, dq
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="gpu", choices=["gpu", "reference"])
    ap.add_argument("--workload", default="C4", choices=sorted(synth.WORKLOADS),
                    help="headline workload (default: the largest single-GPU configuration)")
    ap.add_argument("--configs", default="C2,C3,C5", help="other fine-tuning configurations reported beside the headline ('' = none)")
    ap.add_argument("--min-region-s", type=float, default=1.5, help="repeat the K-step timed region until this much timed work has run")
    ap.add_argument("--min-region-s-configs", type=float, default=1.0)
    ap.add_argument("--geometry", default="GA", choices=["GA", "GB"])
    ap.add_argument("--scale-op", type=int, default=0, choices=[0, 1, 2],
                    help="adapter operator pair: 0 AvgPool & repeat_interleave (the method), 1 truncation & zero padding, "
                         "2 interval sampling & zero fill (Sec. 4 ablation)")
    ap.add_argument("--ref-rows", type=int, default=0, help="token rows per oracle step (bounded sample; 0 = sized for about 45 GF per step)")
    ap.add_argument("--ref-max-steps", type=int, default=3)
    ap.add_argument("--no-extras", action="store_true", help="skip the deploy-path blocks (lowbit, dense_16bit)")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense_16bit block only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of graph replay")
    ap.add_argument("--lowbit-shapes", default="q,up", help="linears of C5 timed in the lowbit extras")
    ap.add_argument("--lowbit-tokens", default="1,16,2048", help="token counts timed in the lowbit extras")
    args = ap.parse_args()
    global SCALE_OP
    SCALE_OP = args.scale_op
    args.warmup = max(args.warmup, 3) if args.impl == "gpu" else args.warmup
    wl = synth.WORKLOADS[args.workload]
    geom = synth.GEOM_A if args.geometry == "GA" else synth.GEOM_B
    if args.impl == "reference":
        run_reference(args, wl, geom)
    else:
        run_gpu(args, wl, geom)


if __name__ == "__main__":
    main()
