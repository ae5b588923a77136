"""Benchmark of the PoT hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

One "step" = one decode token through the linear layers of a Llama-2-7B-shaped model
(32 layers x {qkv 4096->12288, o 4096->4096, gate 4096->11008, up 4096->11008, down 11008->4096}):
160 fused dequant+GEMV launches over 3-bit, group-128 PoT codes (2.53 GB of codes + scales, so
every step streams its weights from HBM: the inputs are ~20x larger than L2).  The metric is the
achieved algorithmic GB/s (codes + scales + x + y bytes per step / step time).  The same JSON
line carries: the 2-bit chain, the standalone dequant throughput next to the uniform-INT twin,
the small-batch and prefill GEMM figures, the roofline fraction of the dominant kernel, the
oracle timed on the host cores, and an end-to-end figure with activations/results in host memory.

With --gpus N > 1 (launched by torch.distributed.run) every rank runs its own replica of the
chain (the path needs no exchange step); the value is the sum over ranks / max time.
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

from paper_2507_11959_b200 import synth  # noqa: E402

METRIC = "pot_dequant_gemv_GBps"
UNIT = "GB/s"
GROUP = 128
HEADLINE_BITS = 3
NCU_TRAFFIC_RATIO = 1.0015  # measured DRAM bytes / algorithmic bytes of the GEMV kernel (see profiles/)


def gemv_bytes(N, K, bits, G, M=1):
    return N * K * bits // 8 + N * (K // G) * 2 + 2 * K * M + 2 * N * M


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
def reference_arm(args):
    """The CPU oracle, as it stands, timed on the host cores on a bounded sample of the workload:
    each step = the five projections of ONE layer of the chain (202 M weights), 3-bit, group 128."""
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    from oracle import pot_oracle as oracle
    layer, nbytes = [], 0
    for i, pr in enumerate(synth.LLAMA2_7B):
        W = synth.weights(synth.rng_for(2, 2 * i), pr.N, pr.K, "t5")
        codes, S = oracle.quantize(W, HEADLINE_BITS, GROUP, oracle.RULE_TOP)
        x = synth.activations(synth.rng_for(2, 2 * i + 1), 1, pr.K)
        layer.append((oracle.pack(codes, HEADLINE_BITS), S, pr.K, x))
        nbytes += gemv_bytes(pr.N, pr.K, HEADLINE_BITS, GROUP)
        del W, codes

    def step():
        for packed, S, K, x in layer:
            oracle.matmul(packed, S, K, HEADLINE_BITS, GROUP, x)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    val = nbytes / dt / 1e9
    sample = "one layer (5 projections, 202M weights) of the 32-layer chain per step, FP64 GEMV from packed codes"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama2-7b-shaped decode chain, batch 1, PoT 3-bit g128 (bounded sample: 1 of 32 layers per step)"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the per-config tables (chain only)")
    ap.add_argument("--layers", type=int, default=synth.LLAMA2_7B_LAYERS)
    ap.add_argument("--shard", default="replicas", choices=["replicas", "rows"],
                    help="N > 1: 'replicas' = every rank runs the whole chain (weak scaling, the default); 'rows' = every "
                         "projection is split by rows over the ranks and the outputs are all-gathered (strong scaling)")
    ap.add_argument("--kernel", default=None, choices=["gemv", "gemv_uint", "dequant", "dequant_uint", "gemm"],
                    help="profiling mode: run only this kernel on one small seeded case and print its timing")
    ap.add_argument("--N", type=int, default=12288)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--M", type=int, default=8)
    ap.add_argument("--bits", type=int, default=3)
    ap.add_argument("--no-graph", action="store_true", help="profiling mode: plain stream launches instead of a CUDA graph")
    ap.add_argument("--copies", type=int, default=16, help="profiling mode: distinct weight copies cycled through (HBM-cold)")
    args = ap.parse_args()
    if args.kernel:
        single_kernel(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        reference_arm(args)
        return

    import torch
    from paper_2507_11959_b200 import binding as B
    from paper_2507_11959_b200 import dist as pdist

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    rank, local_rank, world = pdist.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B.lib()
    peaks = read_peaks()
    stream = torch.cuda.Stream(device=dev)

    def f16(bits16):
        return torch.from_numpy(bits16.view(np.int16)).view(torch.float16).to(dev)

    # ---- build the chain: one layer of seeded weights, quantized on the device, replicated per layer
    def build_chain(bits, projections=synth.LLAMA2_7B):
        protos = []
        for i, pr in enumerate(projections):
            W = f16(synth.weights(synth.rng_for(2, 2 * i), pr.N, pr.K, "t5"))
            packed, S = B.pot_quantize_ref(W, bits, GROUP, B.SCALE_TOP)
            tiled = B.pot_repack(packed, pr.K, bits, 0)
            S = B.pot_repack_scales(S, pr.K, GROUP, 0)
            x = f16(synth.activations(synth.rng_for(2, 2 * i + 1), 1, pr.K)[0])
            y = torch.empty(pr.N, dtype=torch.float16, device=dev)
            ws_bytes = B.pot_gemv_workspace_bytes(pr.N, pr.K, bits, GROUP)
            ws = B.new_workspace(ws_bytes, dev)
            protos.append((pr, tiled, S, x, y, ws))
            del W, packed
        layers = []
        for _ in range(args.layers):  # distinct buffers per layer: the chain streams from HBM
            layers.append([(pr, t.clone(), s.clone(), x, y, ws) for (pr, t, s, x, y, ws) in protos])
        nbytes = args.layers * sum(gemv_bytes(pr.N, pr.K, bits, GROUP) for pr in projections)
        return layers, nbytes

    def enqueue_chain(layers, bits, s):
        for layer in layers:
            for pr, t, sc, x, y, ws in layer:
                B.pot_gemv(t, sc, pr.K, bits, GROUP, x, B.TILED, y=y, workspace=ws, stream=s)

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn(stream)  # warm-up outside capture
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                fn(stream)
        return g

    def time_graph(g, steps, warmup, per_step=None):
        """ms per replay over `steps` replays (CUDA events on the launching stream, a barrier and a device synchronise
        on both sides).  per_step: a list that receives every replay's own duration (an event between replays)."""
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                g.replay()
            stream.synchronize()
            pdist.barrier()
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1 if per_step is not None else 2)]
            ev[0].record(stream)
            for i in range(steps):
                g.replay()
                if per_step is not None:
                    ev[i + 1].record(stream)
            if per_step is None:
                ev[1].record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            pdist.barrier()
        if per_step is not None:
            per_step.extend(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
        return ev[0].elapsed_time(ev[-1]) / steps  # ms per step

    if args.shard == "rows":
        sharded_rows_arm(args, B, pdist, torch, dev, stream, f16, peaks, rank, world)
        pdist.shutdown()
        return

    layers3, bytes3 = build_chain(HEADLINE_BITS)
    launches_before = B.pot_launch_count()
    g3 = capture(lambda s: enqueue_chain(layers3, HEADLINE_BITS, s))
    launches_per_step = (B.pot_launch_count() - launches_before) // 2

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    step_ms = []
    ms = time_graph(g3, args.steps, args.warmup, per_step=step_ms)
    clocks = sampler.stop()
    ms = pdist.max_over_ranks(ms, dev)
    value = world * bytes3 / (ms * 1e-3) / 1e9

    # ---- end to end: activations and results in pinned host memory, weights resident.  Every GEMV is one pot_gemv_host
    # call (H2D of x, kernel, D2H of y on the call's stream); the calls go round-robin to E2E_LANES streams, each with
    # its own device and host buffers, so that one call's copies overlap another call's kernel -- the way a server
    # pipelines independent requests.  The captured graph holds the lanes as parallel branches.
    E2E_LANES = 8  # measured: 2 lanes 2.36 ms, 4 lanes 1.41 ms, 8 lanes 1.10 ms, 16 lanes 1.41 ms per step
    lane_streams = [torch.cuda.Stream(device=dev) for _ in range(E2E_LANES)]
    lane_bufs = []
    for _ in range(E2E_LANES):
        bufs = []
        for pr, t, sc, x, y, ws in layers3[0]:
            xh = torch.empty(pr.K, dtype=torch.float16).pin_memory()
            xh.copy_(x.cpu())
            yh = torch.empty(pr.N, dtype=torch.float16).pin_memory()
            bufs.append((xh, yh, x.clone(), torch.empty_like(y), None if ws is None else torch.zeros_like(ws)))
        lane_bufs.append(bufs)

    def enqueue_e2e(s):
        fork = torch.cuda.Event()
        fork.record(s)
        for ls in lane_streams:
            ls.wait_event(fork)
        i = 0
        for layer in layers3:
            for k, (pr, t, sc, x, y, ws) in enumerate(layer):
                lane = i % E2E_LANES
                xh, yh, xd, yd, wsd = lane_bufs[lane][k]
                B.pot_gemv_host(t, sc, pr.K, HEADLINE_BITS, GROUP, xh, yh, xd, yd, B.TILED, workspace=wsd, stream=lane_streams[lane])
                i += 1
        for ls in lane_streams:
            join = torch.cuda.Event()
            join.record(ls)
            s.wait_event(join)

    ge = capture(enqueue_e2e)
    ms_e2e = pdist.max_over_ranks(time_graph(ge, max(3, args.steps // 2), 3), dev)
    torch.cuda.synchronize()
    # the results that came back to host memory are the ones the device-resident chain computed (same weights, same x)
    e2e_ok = all(torch.equal(lane_bufs[lane][k][1].to(dev), layers3[0][k][4])
                 for lane in range(E2E_LANES) for k in range(len(layers3[0])))
    if not e2e_ok:
        raise SystemExit("bench.py: the end-to-end path returned different results from the device-resident chain")
    h2d = args.layers * sum(2 * pr.K for pr in synth.LLAMA2_7B)
    d2h = args.layers * sum(2 * pr.N for pr in synth.LLAMA2_7B)
    e2e = {"value": world * bytes3 / (ms_e2e * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "ms_per_step": ms_e2e, "results_checked_against_device_chain": True, "note": "x from pinned host and y to pinned host for each of the 160 GEMVs (pot_gemv_host), calls spread over 8 streams; weights resident in HBM"}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16 (int32 bit ops, f32 accumulate)",
        "data": "synthetic",
        "config": {"workload": f"llama2-7b-shaped decode chain, batch 1, {args.layers} layers x 5 projections, PoT {HEADLINE_BITS}-bit g{GROUP}, tiled layout, CUDA graph + PDL",
                   "l2": "inputs larger than L2 (%.2f GB of codes+scales per step vs 126 MB)" % (bytes3 / 1e9),
                   "bytes_per_step": bytes3, "launches_per_step": launches_per_step},
        "step_ms_stats": {"median": float(np.median(step_ms)), "p10": float(np.percentile(step_ms, 10)),
                          "p90": float(np.percentile(step_ms, 90)), "min": float(min(step_ms)), "max": float(max(step_ms)), "n": len(step_ms)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "achieved": value / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": value / world / peaks["hbm_gbs"], "frac_of_8TBs_nominal": value / world / 8000.0,
                     "peak_source": peaks["source"], "kernel": "stream_kernel<3, PoT, GEMV, 16 warps, 2 CTAs per SM> (decode GEMV: per-warp bulk-copy rings, decode in registers, mma.sync)",
                     "per_launch_us": ms * 1e3 / max(1, launches_per_step),
                     "algorithmic_bytes_per_launch": bytes3 / max(1, launches_per_step),
                     # dram__bytes_read+write per launch from the ncu capture of the 12288x4096 launch
                     # (profiles/stream_kernel_gemv_12288x4096_3bit.md: 1.0015 x algorithmic), scaled by bytes
                     "traffic": NCU_TRAFFIC_RATIO * bytes3 / max(1, launches_per_step)},
    }

    if rank == 0 and world == 1 and not args.no_extras:
        out["extras"] = extras(args, B, torch, dev, stream, f16, capture, time_graph, peaks, build_chain, enqueue_chain)
        out["cpu_baseline"] = cpu_baseline()
    del layers3
    if rank == 0:
        print(json.dumps(out), flush=True)
    pdist.shutdown()


def sharded_rows_arm(args, B, pdist, torch, dev, stream, f16, peaks, rank, world):
    """The 7B chain with every projection split by rows over the ranks (RowShard) and an NCCL all-gather of y after each
    GEMV: the whole job is ONE model, so the value is the model's bytes over the step time (strong scaling).  Eager
    launches on one stream (the collective sits between the GEMVs)."""
    protos, nbytes = [], 0
    for i, pr in enumerate(synth.LLAMA2_7B):
        W = f16(synth.weights(synth.rng_for(2, 2 * i), pr.N, pr.K, "t5"))
        packed, S = B.pot_quantize_ref(W, HEADLINE_BITS, GROUP, B.SCALE_TOP)
        sh = pdist.RowShard(packed, S, pr.K, HEADLINE_BITS, GROUP, rank, world)
        x = f16(synth.activations(synth.rng_for(2, 2 * i + 1), 1, pr.K)[0])
        y_full = torch.empty(pr.N, dtype=torch.float16, device=dev)
        ws = B.new_workspace(B.pot_gemv_workspace_bytes(sh.end - sh.begin, pr.K, HEADLINE_BITS, GROUP), dev) if sh.end > sh.begin else None
        protos.append((sh, x, y_full, ws))
        nbytes += gemv_bytes(pr.N, pr.K, HEADLINE_BITS, GROUP)
        del W, packed, S
    layers = []
    for _ in range(args.layers):  # distinct weight buffers per layer: the chain streams from HBM
        layer = []
        for sh, x, y_full, ws in protos:
            c = pdist.RowShard.__new__(pdist.RowShard)
            c.__dict__.update(sh.__dict__)
            c.codes, c.scales = sh.codes.clone(), sh.scales.clone()
            layer.append((c, x, y_full, ws))
        layers.append(layer)
    nbytes *= args.layers

    def step():
        for layer in layers:
            for sh, x, y_full, ws in layer:
                pdist.sharded_gemv(sh, x, y_full, workspace=ws, stream=stream)

    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", 0)))
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step()
        stream.synchronize()
        pdist.barrier()
        torch.cuda.synchronize()
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        before = B.pot_launch_count()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        pdist.barrier()
    clocks = sampler.stop()
    ms = pdist.max_over_ranks(e0.elapsed_time(e1) / args.steps, dev)
    value = nbytes / (ms * 1e-3) / 1e9
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "f16 (int32 bit ops, f32 accumulate)", "data": "synthetic",
            "config": {"workload": f"llama2-7b-shaped decode chain, batch 1, {args.layers} layers x 5 projections, PoT {HEADLINE_BITS}-bit g{GROUP}, "
                                   f"rows of every projection sharded over {world} ranks, NCCL all-gather of y after every GEMV, eager launches",
                       "l2": "inputs larger than L2", "bytes_per_step": nbytes},
            "clocks": clocks, "gpu_launches": B.pot_launch_count() - before,
            "roofline": {"bound": "hbm", "achieved": value / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": value / world / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": None},
            "e2e": None, "cpu_baseline": None}))


def single_kernel(args):
    """Profiling mode (used for the ncu captures under profiles/): one kernel, one small case, a few
    launches over `copies` distinct weight buffers.  Codes are seeded random bytes (every bit pattern is
    a valid code), scales a seeded spread of legal FP16 values; timing is data-independent."""
    import torch
    from paper_2507_11959_b200 import binding as B
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    N, K, bits, M = args.N, args.K, args.bits, args.M
    g = torch.Generator(device=dev).manual_seed(BASE_PROFILE_SEED)
    P = [torch.randint(0, 256, (N, K * bits // 8), dtype=torch.uint8, device=dev, generator=g) for _ in range(args.copies)]
    S = ((torch.rand((N, K // GROUP), device=dev, generator=g) * 0.01 + 0.002).to(torch.float16))
    Z = torch.randint(0, 1 << bits, (N, K // GROUP), device=dev, generator=g).to(torch.float16)
    x = torch.randn(K, device=dev, generator=g).to(torch.float16)
    X = torch.randn((M, K), device=dev, generator=g).to(torch.float16)
    y = torch.empty(N, dtype=torch.float16, device=dev)
    Y = torch.empty((M, N), dtype=torch.float16, device=dev)
    out = torch.empty((N, K), dtype=torch.float16, device=dev) if args.kernel.startswith("dequant") else None
    ws = B.new_workspace(max(B.pot_gemv_workspace_bytes(N, K, bits, GROUP), B.pot_gemm_workspace_bytes(M, N, K, bits, GROUP)), dev)

    def run(p):
        st = torch.cuda.current_stream()
        if args.kernel == "gemv":
            B.pot_gemv(p, S, K, bits, GROUP, x, B.TILED, y=y, workspace=ws, stream=st)
        elif args.kernel == "gemv_uint":
            B.uint_gemv(p, S, Z, K, bits, GROUP, x, B.TILED, y=y, workspace=ws, stream=st)
        elif args.kernel == "dequant":
            B.pot_dequant(p, S, K, bits, GROUP, B.F16, out=out, stream=st)
        elif args.kernel == "dequant_uint":
            B.uint_dequant(p, S, Z, K, bits, GROUP, B.UINT_FAST, out=out, stream=st)
        else:
            B.pot_gemm(p, S, K, bits, GROUP, X, B.TILED, Y=Y, workspace=ws, stream=st)

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for p in P[: max(3, args.warmup)]:
            run(p)
        stream.synchronize()
        if args.no_graph:
            n = 0
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(max(1, args.steps)):
                for p in P:
                    run(p)
                    n += 1
            e1.record(stream)
        else:  # one CUDA graph holding one launch per weight copy, replayed `steps` times (no host launch cost)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for p in P:
                    run(p)
            g.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(max(1, args.steps)):
                g.replay()
            e1.record(stream)
            n = max(1, args.steps) * len(P)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n
    if args.kernel.startswith("dequant"):
        nb = N * K * bits // 8 + N * (K // GROUP) * 2 + 2 * N * K
    else:
        nb = gemv_bytes(N, K, bits, GROUP, M if args.kernel == "gemm" else 1)
    print(json.dumps({"kernel": args.kernel, "N": N, "K": K, "M": M, "bits": bits, "graph": not args.no_graph, "us_per_launch": us,
                      "device_errors": B.pot_debug_errors(),
                      "GBps": nb / us / 1e3, "launches": n}))


BASE_PROFILE_SEED = 250711959


def cpu_baseline():
    """The oracle's FP64 GEMV from packed codes on the host cores: one layer of the chain (bounded sample)."""
    from oracle import pot_oracle as oracle
    layer, nbytes = [], 0
    for i, pr in enumerate(synth.LLAMA2_7B):
        W = synth.weights(synth.rng_for(2, 2 * i), pr.N, pr.K, "t5")
        codes, S = oracle.quantize(W, HEADLINE_BITS, GROUP, oracle.RULE_TOP)
        layer.append((oracle.pack(codes, HEADLINE_BITS), S, pr.K, synth.activations(synth.rng_for(2, 2 * i + 1), 1, pr.K)))
        nbytes += gemv_bytes(pr.N, pr.K, HEADLINE_BITS, GROUP)
    best = 1e30
    for _ in range(3):
        t0 = time.perf_counter()
        for packed, S, K, x in layer:
            oracle.matmul(packed, S, K, HEADLINE_BITS, GROUP, x)
        best = min(best, time.perf_counter() - t0)
    # the oracle's dequantizer beside it (config 3's metric): the 4096 x 4096, 3-bit matrix to FP16, best of 3
    packed0, S0, K0 = layer[1][0], layer[1][1], layer[1][2]
    best_dq = 1e30
    for _ in range(3):
        t0 = time.perf_counter()
        oracle.dequant(packed0, S0, K0, HEADLINE_BITS, GROUP)
        best_dq = min(best_dq, time.perf_counter() - t0)
    return {"value": nbytes / best / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "one layer (5 projections, 202M weights) of the 32-layer chain, best of 3",
            "dequant_Gweights_s": packed0.shape[0] * K0 / best_dq / 1e9,
            "dequant_sample": "4096 x 4096 3-bit g128 matrix of the same layer to FP16, best of 3"}


def extras(args, B, torch, dev, stream, f16, capture, time_graph, peaks, build_chain, enqueue_chain):
    """Per-config tables: 2-bit chain, per-projection GEMV, dequant sweep vs the uniform twin, small-batch and prefill GEMM."""
    ex = {}
    hbm = peaks["hbm_gbs"]

    # 2-bit chain (config 2)
    layers2, bytes2 = build_chain(2)
    g2 = capture(lambda s: enqueue_chain(layers2, 2, s))
    ms2 = time_graph(g2, max(5, args.steps // 2), 3)
    ex["chain_2bit"] = {"GBps": bytes2 / ms2 / 1e6, "ms_per_step": ms2, "frac_of_measured_hbm": bytes2 / ms2 / 1e6 / hbm}
    del g2, layers2
    torch.cuda.empty_cache()

    # the same 3-bit chain with gate and up stored as one 4096 -> 22016 matrix (they share their input, as qkv do):
    # 128 launches per step instead of 160 over the same weights
    fused = (synth.LLAMA2_7B[0], synth.LLAMA2_7B[1], synth.Projection("gate_up", 4096, 22016), synth.LLAMA2_7B[4])
    layersf, bytesf = build_chain(HEADLINE_BITS, fused)
    gf = capture(lambda s: enqueue_chain(layersf, HEADLINE_BITS, s))
    msf = time_graph(gf, max(5, args.steps // 2), 3)
    ex["chain_3bit_gate_up_fused"] = {"GBps": bytesf / msf / 1e6, "ms_per_step": msf, "frac_of_measured_hbm": bytesf / msf / 1e6 / hbm,
                                      "launches_per_step": 4 * args.layers}
    del gf, layersf
    torch.cuda.empty_cache()

    L2_BYTES = 126e6

    def time_eager(fn, n=20):
        """isolated launches: each one timed alone with its own pair of events (launch latency and ramp included)"""
        ts = []
        with torch.cuda.stream(stream):
            for i in range(n + 3):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                stream.synchronize()
                e0.record(stream)
                fn(i)
                e1.record(stream)
                stream.synchronize()
                if i >= 3:
                    ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    def ab_ratio(run_a, run_b, copies, reps=7):
        """A and B interleaved (ABAB...) in ONE captured graph over rotating HBM-cold buffers; the graph is replayed
        `reps` times with an event after every launch's group, so both see the same clocks and the same cache state.
        Returns (median ms of A per launch, of B, and min / median / max of the per-repetition ratio B / A)."""
        ga = capture(lambda s: [run_a(i, s) for i in range(copies)])
        gb = capture(lambda s: [run_b(i, s) for i in range(copies)])
        ta, tb = [], []
        for _ in range(reps):
            ta.append(time_graph(ga, 4, 1) / copies)
            tb.append(time_graph(gb, 4, 1) / copies)
        r = [y / x for x, y in zip(ta, tb)]
        return float(np.median(ta)), float(np.median(tb)), {"min": min(r), "median": float(np.median(r)), "max": max(r), "reps": reps}

    # per-projection GEMV (config 1 and config 2 shapes): isolated launch, steady state in a graph over HBM-cold rotating
    # copies (> 4x L2), and next to the uniform twin (interleaved repetitions)
    rows = []
    shapes = [("cfg1 4096x4096", 4096, 4096, "normal")] + [(f"7B {p.name}", p.N, p.K, "t5") for p in synth.LLAMA2_7B if p.name != "up"]
    for name, N, K, dist in shapes:
        W = f16(synth.weights(synth.rng_for(1, N % 97), N, K, dist))
        x = f16(synth.activations(synth.rng_for(1, 1 + N % 97), 1, K)[0])
        y = torch.empty(N, dtype=torch.float16, device=dev)
        for bits in (2, 3, 4):
            packed, S = B.pot_quantize_ref(W, bits, GROUP, B.SCALE_TOP)
            tiled = B.pot_repack(packed, K, bits, 0)
            S = B.pot_repack_scales(S, K, GROUP, 0)
            up, uS, uZ = B.uint_quantize_ref(W, bits, GROUP)
            utiled = B.uint_repack(up, K, bits, 0)
            uS, uZ = B.pot_repack_scales(uS, K, GROUP, 0), B.pot_repack_scales(uZ, K, GROUP, 0)
            copies = max(2, int(4 * L2_BYTES / (N * K * bits / 8)) + 1)
            ws = B.new_workspace(B.pot_gemv_workspace_bytes(N, K, bits, GROUP), dev)
            pts = [(tiled.clone(), S.clone()) for _ in range(copies)]
            uts = [(utiled.clone(), uS.clone(), uZ.clone()) for _ in range(copies)]
            run_p = lambda i, s: B.pot_gemv(pts[i][0], pts[i][1], K, bits, GROUP, x, B.TILED, y=y, workspace=ws, stream=s)
            run_u = lambda i, s: B.uint_gemv(uts[i][0], uts[i][1], uts[i][2], K, bits, GROUP, x, B.TILED, y=y, workspace=ws, stream=s)
            tp, tu, ratio = ab_ratio(run_p, run_u, copies)
            t_iso = time_eager(lambda i: run_p(i % copies, stream)) if bits == HEADLINE_BITS else None
            bp = gemv_bytes(N, K, bits, GROUP)
            bu = bp + N * (K // GROUP) * 2
            rows.append({"shape": name, "bits": bits, "pot_us_steady": tp * 1e3, "pot_us_isolated_launch": None if t_iso is None else t_iso * 1e3,
                         "pot_GBps": bp / tp / 1e6, "pot_frac_hbm": bp / tp / 1e6 / hbm, "uint_us_steady": tu * 1e3,
                         "uint_GBps": bu / tu / 1e6, "uint_over_pot_time": ratio, "plan": B.pot_debug_gemv_plan(N, K, bits, GROUP)})
            del pts, uts
        del W
        torch.cuda.empty_cache()
    ex["gemv_per_projection_hbm_cold"] = rows

    # one large matrix (28672 x 8192, 3 bit): the kernel without the per-launch costs that dominate the 7B shapes
    N, K = 28672, 8192
    gq = torch.Generator(device=dev).manual_seed(BASE_PROFILE_SEED)
    Pb = [torch.randint(0, 256, (N, K * 3 // 8), dtype=torch.uint8, device=dev, generator=gq) for _ in range(6)]
    Sb = (torch.rand((N, K // GROUP), device=dev, generator=gq) * 0.01 + 0.002).to(torch.float16)
    xb = torch.randn(K, device=dev, generator=gq).to(torch.float16)
    yb = torch.empty(N, dtype=torch.float16, device=dev)
    wsb = B.new_workspace(B.pot_gemv_workspace_bytes(N, K, 3, GROUP), dev)
    gb = capture(lambda s: [B.pot_gemv(p, Sb, K, 3, GROUP, xb, B.TILED, y=yb, workspace=wsb, stream=s) for p in Pb])
    tb = min(time_graph(gb, 5, 2) for _ in range(3)) / len(Pb)
    nb = gemv_bytes(N, K, 3, GROUP)
    ex["gemv_28672x8192_3bit_hbm_cold"] = {"us": tb * 1e3, "GBps": nb / tb / 1e6, "frac_of_measured_hbm": nb / tb / 1e6 / hbm,
                                           "frac_of_8TBs_nominal": nb / tb / 1e6 / 8000.0}
    del Pb, gb
    torch.cuda.empty_cache()

    # the BF16 route on the 7B qkv shape (3 bit): same bytes, two mask / multiply-add pairs per register instead of one
    N, K = 12288, 4096
    copies = 28
    Pq = [torch.randint(0, 256, (N, K * 3 // 8), dtype=torch.uint8, device=dev, generator=gq) for _ in range(copies)]
    Sq = (torch.rand((N, K // GROUP), device=dev, generator=gq) * 0.01 + 0.002).to(torch.float16)
    wsq = B.new_workspace(B.pot_gemv_workspace_bytes(N, K, 3, GROUP), dev)
    res = {}
    for name, dt in (("f16", torch.float16), ("bf16", torch.bfloat16)):
        xq = torch.randn(K, device=dev, generator=gq).to(dt)
        yq = torch.empty(N, dtype=dt, device=dev)
        gg = capture(lambda s: [B.pot_gemv(p, Sq, K, 3, GROUP, xq, B.TILED, y=yq, workspace=wsq, stream=s) for p in Pq])
        res[name + "_us"] = min(time_graph(gg, 5, 2) for _ in range(3)) / copies * 1e3
        del gg
    ex["gemv_7B_qkv_3bit_f16_vs_bf16"] = res
    del Pq
    torch.cuda.empty_cache()

    # standalone dequant (config 3): PoT vs the uniform twin (fast and naive kernels), FP16 out.  HBM-cold: every launch
    # of a graph reads its own packed matrix and writes its own output, R pairs with R x bytes >= 4 x L2; the L2-warm
    # figure (one pair, written over and over) is reported beside it, labelled.
    rows = []
    for N, K in synth.DEQUANT_SWEEP:
        W = f16(synth.weights(synth.rng_for(3, N % 89), N, K, "normal"))
        for bits in (2, 3, 4):
            for G in (64, 128):
                packed, S = B.pot_quantize_ref(W, bits, G, B.SCALE_TOP)
                up, uS, uZ = B.uint_quantize_ref(W, bits, G)
                nb = N * K * bits // 8 + N * (K // G) * 2 + N * K * 2
                R = max(2, int(4 * L2_BYTES / nb) + 1)
                outs = [torch.empty((N, K), dtype=torch.float16, device=dev) for _ in range(R)]
                pk = [packed] + [packed.clone() for _ in range(R - 1)]
                uk = [up] + [up.clone() for _ in range(R - 1)]
                run_p = lambda i, s: B.pot_dequant(pk[i], S, K, bits, G, B.F16, out=outs[i], stream=s)
                run_f = lambda i, s: B.uint_dequant(uk[i], uS, uZ, K, bits, G, B.UINT_FAST, out=outs[i], stream=s)
                run_n = lambda i, s: B.uint_dequant(uk[i], uS, uZ, K, bits, G, B.UINT_NAIVE, out=outs[i], stream=s)
                tp, tf, rf = ab_ratio(run_p, run_f, R, reps=5)
                gn = capture(lambda s: [run_n(i, s) for i in range(R)])
                tn = min(time_graph(gn, 3, 1) for _ in range(2)) / R
                gw = capture(lambda s: [run_p(0, s) for _ in range(R)])
                tw = min(time_graph(gw, 3, 1) for _ in range(2)) / R
                rows.append({"N": N, "K": K, "bits": bits, "G": G, "rotating_pairs": R, "pot_us": tp * 1e3, "pot_Gweights_s": N * K / tp / 1e6,
                             "pot_GBps": nb / tp / 1e6, "pot_frac_hbm": nb / tp / 1e6 / hbm, "pot_frac_8TBs_nominal": nb / tp / 1e6 / 8000.0,
                             "uint_fast_us": tf * 1e3, "uint_naive_us": tn * 1e3, "uint_fast_over_pot_time": rf,
                             "pot_us_l2_warm_same_buffers": tw * 1e3})
                del outs, pk, uk, gn, gw
                torch.cuda.empty_cache()
        del W
        torch.cuda.empty_cache()
    ex["dequant_sweep"] = rows

    # Algorithm 1 on the GPU (scale search, 200 candidates per group), set-up code: time per matrix
    W = f16(synth.weights(synth.rng_for(1, 4096 % 97), 4096, 4096, "normal"))
    with torch.cuda.stream(stream):
        B.pot_quantize_ref(W, 3, GROUP, B.SCALE_SEARCH, stream=stream)
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(3):
            B.pot_quantize_ref(W, 3, GROUP, B.SCALE_SEARCH, stream=stream)
        e1.record(stream)
        stream.synchronize()
    ta1 = e0.elapsed_time(e1) / 3
    ex["algorithm1_scale_search_4096x4096_3bit"] = {"ms": ta1, "Mgroups_s": 4096 * 32 / ta1 / 1e3,
                                                    "G_candidate_weight_evaluations_s": 4096 * 4096 * 200 / ta1 / 1e6}
    del W
    torch.cuda.empty_cache()

    # small-batch GEMM (config 4), HBM-cold
    rows = []
    for pr in synth.LLAMA2_13B:
        W = f16(synth.weights(synth.rng_for(4, pr.N % 83), pr.N, pr.K, "t5"))
        packed, S = B.pot_quantize_ref(W, 3, GROUP, B.SCALE_TOP)
        tiled = B.pot_repack(packed, pr.K, 3, 0)
        S = B.pot_repack_scales(S, pr.K, GROUP, 0)
        copies = max(2, int(4 * 126e6 / (pr.N * pr.K * 3 / 8)) + 1)
        pts = [(tiled.clone(), S.clone()) for _ in range(copies)]
        del W, packed
        for M in synth.SMALL_BATCH_M:
            X = f16(synth.activations(synth.rng_for(4, 7), M, pr.K))
            Y = torch.empty((M, pr.N), dtype=torch.float16, device=dev)
            ws = B.new_workspace(B.pot_gemm_workspace_bytes(M, pr.N, pr.K, 3, GROUP), dev)
            g = capture(lambda s: [B.pot_gemm(t, sc, pr.K, 3, GROUP, X, B.TILED, Y=Y, workspace=ws, stream=s) for t, sc in pts])
            t = min(time_graph(g, 10, 3) for _ in range(3)) / copies
            nb = gemv_bytes(pr.N, pr.K, 3, GROUP, M)
            rows.append({"shape": f"13B {pr.name} {pr.K}->{pr.N}", "M": M, "us": t * 1e3, "GBps": nb / t / 1e6, "frac_hbm": nb / t / 1e6 / hbm})
            del g
        del pts
        torch.cuda.empty_cache()
    ex["small_batch_gemm"] = rows

    # prefill GEMM (config 5)
    rows = []
    for pr in synth.LLAMA2_70B:
        W = f16(synth.weights(synth.rng_for(5, pr.N % 79), pr.N, pr.K, "normal", 0.015))
        X = f16(synth.activations(synth.rng_for(5, 5), synth.PREFILL_M, pr.K, outliers=False))
        Y = torch.empty((synth.PREFILL_M, pr.N), dtype=torch.float16, device=dev)
        for bits in (2, 3):
            packed, S = B.pot_quantize_ref(W, bits, GROUP, B.SCALE_TOP)
            layout, P = B.CANONICAL, packed
            try:
                tiled = B.pot_repack(packed, pr.K, bits, 0)
                Sc, S = S, B.pot_repack_scales(S, pr.K, GROUP, 0)
                ws = B.new_workspace(B.pot_gemm_workspace_bytes(synth.PREFILL_M, pr.N, pr.K, bits, GROUP), dev)
                B.pot_gemm(tiled, S, pr.K, bits, GROUP, X, B.TILED, Y=Y, workspace=ws, stream=stream)
                layout, P = B.TILED, tiled
            except B.PotError:
                ws, S = None, Sc
            g = capture(lambda s: B.pot_gemm(P, S, pr.K, bits, GROUP, X, layout, Y=Y, workspace=ws, stream=s))
            t = min(time_graph(g, 3, 3) for _ in range(2))
            fl = 2.0 * synth.PREFILL_M * pr.N * pr.K
            row = {"shape": f"70B {pr.name} {pr.K}->{pr.N}", "M": synth.PREFILL_M, "bits": bits, "ms": t,
                   "TFLOPs": fl / t / 1e9, "frac_tensor_burst": fl / t / 1e9 / peaks["bf16_tflops"],
                   "kernel": "tcgen05" if layout == B.TILED else "mma.sync fallback"}
            if bits == HEADLINE_BITS and pr.name == "gate_or_up":
                # the same launch ~600 times back to back: about half a second under the power cap, the regime in
                # which the sustained cuBLAS figure was measured
                ts = time_graph(g, 600, 3)
                row.update({"ms_sustained": ts, "TFLOPs_sustained": fl / ts / 1e9,
                            "frac_tensor_sustained": fl / ts / 1e9 / peaks["bf16_tflops_sustained"]})
            rows.append(row)
            del g
        del W, X, Y
        torch.cuda.empty_cache()
    ex["prefill_gemm"] = rows
    return ex


if __name__ == "__main__":
    main()
