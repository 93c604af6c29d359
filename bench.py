#!/usr/bin/env python
"""Benchmark of the BitNet a4.8 BitLinear forward on B200.

One step = the seven BitLinears of one 7B-shape transformer layer over 16384
tokens (prefill of 4096 tokens x batch 4): the per-token quantisers (INT4 for
the q/k/v and gate/up inputs, top-K 50 % + INT8 for the o and down inputs)
followed by the packed-ternary contractions and their rescale.  The headline
value is dense-equivalent TOPS (2*M*N*K summed over the seven projections,
divided by the step time, quantisers included).  The same JSON line also
carries the batch-1 decode figure (GB/s of packed weight bytes streamed over
every matrix of the 32-layer model), block tokens/s, the roofline of the
dominant kernel, the end-to-end figure with host buffers, and the CPU oracle
timed on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

For N > 1 launch with torch.distributed.run; every rank runs an independent
replica (tokens shard with no exchange), so scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

# 7B shape (model-configuration table of the paper): hidden 4096, GLU 11008, 32 heads, 32 layers
H, F, NH, LAYERS = 4096, 11008, 32, 32
M_PREFILL = 16384  # 4096 tokens x batch 4
EPS = 1e-5
PROJ = (("q", H, H, "int4"), ("k", H, H, "int4"), ("v", H, H, "int4"), ("o", H, H, "topk"),
        ("gate", F, H, "int4"), ("up", F, H, "int4"), ("down", H, F, "topk"))
STEP_OPS = sum(2 * M_PREFILL * n * k for _, n, k, _ in PROJ)

# DRAM bytes per launch of the dominant kernel from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum).
# Capture: profiles/gemm_pair_prefill_M4096_N11008_K4096.md (150.9 MB of DRAM traffic against 208.5 MB of
# algorithmic bytes at M=4096, part of the output still in L2 at kernel end), scaled to the mean algorithmic bytes
# of the seven launches of a step at M=16384 (488 MB): traffic grows with M like the algorithmic bytes do.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 3.53e8


def library_int8_tops(dev, stream):
    """Dense int8 GEMM of the vendor library on this GPU, as a second reference beside the measured bf16 figure."""
    try:
        n = 8192
        a = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=dev)
        b = torch.randint(-1, 2, (n, n), dtype=torch.int8, device=dev).t()  # column-major second operand
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        e0.record(stream)
        for _ in range(reps):
            torch._int_mm(a, b)
        e1.record(stream)
        torch.cuda.synchronize()
        return 2.0 * n ** 3 / (e0.elapsed_time(e1) / reps * 1e-3) / 1e12
    except Exception:  # not every build has the int8 library path
        return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.uuid = None
        try:
            self.uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid)
        except Exception:
            pass
        self.proc, self.out = None, None

    def start(self):
        try:
            self.out = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"]
            if self.uuid:
                cmd += ["-i", self.uuid]
            self.proc = subprocess.Popen(cmd, stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the two wall-clock times (all samples under load if none fall inside)."""
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.flush()
        self.out.seek(0)
        rows = []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.out.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]),
                             [n for n, v in zip(names, parts[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        window = "timed region"
        if not inside:  # region shorter than the sampling period: fall back to every sample taken under load
            inside, window = rows, "whole run (timed region shorter than one sample period)"
        sm = [r[1] for r in inside]
        mx = [r[2] for r in inside]
        power = [r[3] for r in inside]
        reasons = set(n for r in inside for n in r[4])
        try:
            os.unlink(self.out.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = sorted(s for s, p in zip(sm, power) if p >= 0.5 * max(power)) or sorted(sm)
        return {"sm_mhz": busy[len(busy) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power), "window": window}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# --------------------------------------------------------------------------- reference arm (CPU oracle)
_ORACLE_WEIGHTS = {}


def oracle_weights(oracle, seed=4):
    """Ternarised weights of one 7B-shape layer (set-up, done once: not part of a step)."""
    from paper_2411_04965_b200 import synth
    if seed not in _ORACLE_WEIGHTS:
        _ORACLE_WEIGHTS[seed] = {name: oracle.ternarise(synth.ternary_latents(n, k, seed=100 + i).numpy(), EPS)
                                 for i, (name, n, k, _) in enumerate(PROJ)}
    return _ORACLE_WEIGHTS[seed]


def oracle_layer_sample(oracle, n_tokens, nthreads, seed=4):
    """The seven BitLinears of one 7B-shape layer on n_tokens tokens with the CPU oracle; returns seconds."""
    from paper_2411_04965_b200 import synth
    xh = synth.gaussian_outlier_activations(n_tokens, H, seed).numpy()
    sh = synth.student_t3(n_tokens, H, seed + 1).numpy()
    sf = synth.student_t3(n_tokens, F, seed + 2).numpy()
    rng_w = oracle_weights(oracle, seed)
    t0 = time.perf_counter()
    q4, d4 = oracle.quant_int4(xh, EPS, nthreads=nthreads)
    for name in ("q", "k", "v"):
        oracle.linear(q4, d4, *rng_w[name], nthreads=nthreads, want_acc=False)
    c8, d8, _ = oracle.topk_quant_int8(sh, H // 2, EPS, nthreads=nthreads)
    oracle.linear(c8, d8, *rng_w["o"], nthreads=nthreads, want_acc=False)
    q4, d4 = oracle.quant_int4(xh, EPS, nthreads=nthreads)
    for name in ("gate", "up"):
        oracle.linear(q4, d4, *rng_w[name], nthreads=nthreads, want_acc=False)
    c8, d8, _ = oracle.topk_quant_int8(sf, F // 2, EPS, nthreads=nthreads)
    oracle.linear(c8, d8, *rng_w["down"], nthreads=nthreads, want_acc=False)
    return time.perf_counter() - t0


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    from oracle import oracle_a48 as oracle
    oracle.build()
    cores = len(os.sched_getaffinity(0))
    # size the per-step sample so that warm-up + steps stay near two minutes of CPU work
    per_tok = oracle_layer_sample(oracle, 16, cores) / 16.0
    budget_s = 120.0 / max(1, args.steps + min(args.warmup, 1))
    n_tok = int(max(4, min(2048, budget_s / per_tok)))
    for _ in range(min(args.warmup, 1)):
        oracle_layer_sample(oracle, n_tok, cores)
    times = [oracle_layer_sample(oracle, n_tok, cores) for _ in range(args.steps)]
    t = sum(times) / len(times)
    tops = STEP_OPS * (n_tok / M_PREFILL) / t / 1e12
    sample = f"{n_tok} of {M_PREFILL} tokens through the 7 BitLinears of one layer per step"
    line = {
        "impl": "reference", "metric": "bitlinear_prefill_tops_7b", "value": tops, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64 accumulators, float64 scales", "data": "synthetic",
        "config": {"workload": "7B-shape layer (hidden 4096, GLU 11008): 7 BitLinears incl. quantisers, "
                               "prefill 4096 tokens x batch 4 = 16384 tokens (bounded sample per step)",
                   "sample": sample},
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- replicas (N > 1)
class Replicas:
    """The only cross-rank steps of the benchmark: a barrier, and the slowest rank's time.

    Every rank runs an independent replica (tokens shard with no exchange); the job's throughput is the work
    of all ranks divided by the slowest rank's time.  Backend "nccl" on GPUs, "gloo" in the CPU tests.
    """

    def __init__(self, world, backend="nccl", device=None):
        self.world, self.device = world, device
        if world > 1:
            import torch.distributed as dist
            self.dist = dist
            if not dist.is_initialized():
                kw = {"device_id": device} if backend == "nccl" else {}
                dist.init_process_group(backend, **kw)

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()

    def max_ms(self, ms):
        if self.world == 1:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_value(self, units_per_rank, ms_per_step_max):
        """Whole-job throughput: all ranks' units per second of the slowest rank's step."""
        return units_per_rank * self.world / (ms_per_step_max * 1e-3)

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


# --------------------------------------------------------------------------- our arm
class Layer:
    """Packed weights of one 7B-shape layer plus resident activation buffers."""

    def __init__(self, a48, dev, seed, layouts):
        from paper_2411_04965_b200 import synth
        self.w = {}
        for i, (name, n, k, _) in enumerate(PROJ):
            lat = synth.ternary_latents(n, k, seed=seed * 16 + i, device=dev)
            self.w[name] = a48.pack_ternary(lat, EPS, layouts)
            del lat
        torch.cuda.synchronize()


def run_ours(args):
    from paper_2411_04965_b200 import binding as a48
    from paper_2411_04965_b200 import build as a48_build
    from paper_2411_04965_b200 import synth
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the BitLinear path has no CPU fallback")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    reps = Replicas(world, "nccl", dev)
    if rank == 0:
        a48_build.build()
    reps.barrier()
    a48.lib()
    peaks = load_peaks()
    M = M_PREFILL
    stream = torch.cuda.current_stream()

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    max_over_ranks = reps.max_ms

    # ---- resident inputs: larger than L2 (268 MB + 268 MB + 721 MB of fp32 activations per step)
    layer = Layer(a48, dev, seed=4 + rank, layouts=a48.LAYOUT_ALL)
    x_h = synth.gaussian_outlier_activations(M, H, seed=40 + rank, device=dev)
    s_h = synth.student_t3(M, H, seed=41 + rank, device=dev)
    s_f = synth.student_t3(M, F, seed=42 + rank, device=dev)
    codes_h = torch.empty(M, H, dtype=torch.int8, device=dev)
    codes_f = torch.empty(M, F, dtype=torch.int8, device=dev)
    scale = torch.empty(M, dtype=torch.float32, device=dev)
    y_h = torch.empty(M, H, dtype=torch.float32, device=dev)
    y_f = torch.empty(M, F, dtype=torch.float32, device=dev)
    gemm_events = []

    def gemm(name, codes, kind, out, record):
        if record:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
        a48.linear(layer.w[name], codes, scale, kind, a48.ALGO_AUTO, Y=out)
        if record:
            e1.record(stream)
            gemm_events.append((name, e0, e1))

    def step(record=False):
        a48.quant_int4(x_h, EPS, codes_h, scale)
        for name in ("q", "k", "v"):
            gemm(name, codes_h, a48.ACT_INT4, y_h, record)
        a48.topk_quant_int8(s_h, H // 2, EPS, codes_h, scale)
        gemm("o", codes_h, a48.ACT_TOPK_INT8, y_h, record)
        a48.quant_int4(x_h, EPS, codes_h, scale)
        for name in ("gate", "up"):
            gemm(name, codes_h, a48.ACT_INT4, y_f, record)
        a48.topk_quant_int8(s_f, F // 2, EPS, codes_f, scale)
        gemm("down", codes_f, a48.ACT_TOPK_INT8, y_h, record)
        return 11  # kernel launches of this library per step

    sampler = ClockSampler(dev)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin = time.time()
    e0.record(stream)
    launches = 0
    for _ in range(args.steps):
        launches += step(record=True)
    e1.record(stream)
    barrier()
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end)
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    ms_per_step = ms_total / args.steps
    tops = reps.job_value(STEP_OPS, ms_per_step) / 1e12

    gemm_ms = sum(a.elapsed_time(b) for _, a, b in gemm_events)
    gemm_ops = sum(2 * M * n * k for name, _, _ in gemm_events for pn, n, k, _ in PROJ if pn == name)
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12
    # nominal int8:bf16 ratio of 2 on the measured bf16 figure: sustained for a region of a second or more, else burst
    peak_kind = "bf16_tflops_sustained" if ms_total >= 1000.0 else "bf16_tflops"
    int8_peak = 2.0 * peaks[peak_kind]
    roofline = {"bound": "tensor", "achieved": achieved, "peak": int8_peak, "unit": "TOPS",
                "frac": achieved / int8_peak, "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                "kernel": "BitLinear contraction (prefill)", "launches": len(gemm_events),
                "avg_launch_ms": gemm_ms / len(gemm_events),
                "peak_source": f"2 x {peak_kind} of {peaks['source']} peaks (no int8 peak is measured; nominal int8:bf16 = 2)",
                "timed_region_ms": ms_total}
    lib = library_int8_tops(dev, stream) if rank == 0 else None
    if lib:
        roofline["library_int8_tops"] = lib
        roofline["library_int8_note"] = "torch._int_mm (vendor int8 GEMM) 8192^3, 20 calls, same GPU, outside the timed region"

    # ---- end to end with host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.skip_e2e:
        xh_host = x_h.cpu().pin_memory()
        sh_host = s_h.cpu().pin_memory()
        sf_host = s_f.cpu().pin_memory()
        calls = (("q", xh_host, a48.ACT_INT4, 0), ("k", xh_host, a48.ACT_INT4, 0), ("v", xh_host, a48.ACT_INT4, 0),
                 ("o", sh_host, a48.ACT_TOPK_INT8, H // 2), ("gate", xh_host, a48.ACT_INT4, 0),
                 ("up", xh_host, a48.ACT_INT4, 0), ("down", sf_host, a48.ACT_TOPK_INT8, F // 2))
        outs = {name: torch.empty(M, layer.w[name].N, dtype=torch.float32).pin_memory() for name, *_ in calls}
        ws_bytes = max(a48.bitlinear_host_workspace_bytes(layer.w[n], M) for n, *_ in PROJ)
        # three streams, each with its own workspace: the upload of one call, the kernels of another and the
        # download of a third run at the same time (every call still uploads its input and downloads its output)
        e2e_streams = [torch.cuda.Stream(device=dev) for _ in range(3)]
        wss = [torch.zeros(ws_bytes, dtype=torch.uint8, device=dev) for _ in e2e_streams]

        def step_host():
            for i, (name, xin, kind, k) in enumerate(calls):
                j = i % len(e2e_streams)
                a48.bitlinear_host_async(layer.w[name], xin, outs[name], kind, k, EPS, wss[j], stream=e2e_streams[j])
            for st_ in e2e_streams:
                st_.synchronize()

        step_host()
        barrier()
        n_e2e = max(1, min(args.steps, 3))
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            step_host()
        barrier()
        dt = max_over_ranks((time.perf_counter() - t0) * 1e3) / n_e2e
        h2d = 6 * M * H * 4 + M * F * 4
        d2h = 5 * M * H * 4 + 2 * M * F * 4
        e2e = {"value": STEP_OPS * world / (dt * 1e-3) / 1e12, "unit": "TOPS", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": dt, "steps": n_e2e,
               "api": "bitnet_a48_bitlinear_host_async on 3 streams, pinned host buffers, stream sync per step"}
        del xh_host, sh_host, sf_host, outs, wss

    # ---- batch-1 decode over every matrix of the model (distinct buffers >> L2)
    decode = None
    if not args.skip_decode:
        decode = bench_decode(a48, synth, dev, stream, peaks, rank)

    # ---- block forward tokens/s
    block = None
    if not args.skip_block:
        block = bench_block(a48, synth, dev, stream, layer)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        from oracle import oracle_a48 as oracle
        oracle.build()
        cores = len(os.sched_getaffinity(0))
        n_tok = 2048
        t = oracle_layer_sample(oracle, n_tok, cores)
        cpu_baseline = {"value": STEP_OPS * (n_tok / M) / t / 1e12, "unit": "TOPS", "cores": cores, "kind": "oracle",
                        "sample": f"{n_tok} of {M} tokens through the 7 BitLinears of one 7B-shape layer, {t:.1f} s"}

    if rank == 0:
        line = {
            "metric": "bitlinear_prefill_tops_7b", "value": tops, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x int2 -> int32 (scales fp64/fp32)", "data": "synthetic",
            "config": {"workload": "7B-shape layer (hidden 4096, GLU 11008): 7 BitLinears incl. quantisers, "
                                   "prefill 4096 tokens x batch 4 = 16384 tokens",
                       "l2": "inputs larger than L2 (1.26 GB of fp32 activations + 1.3 GB of outputs per step)",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "e2e": e2e,
            "cpu_baseline": cpu_baseline, "decode": decode, "block": block,
        }
        print(json.dumps(line))
    reps.close()


def bench_decode(a48, synth, dev, stream, peaks, rank):
    """BitLinear chain over all 7 x 32 matrices of the 7B shape, one CUDA graph per token count (1, 8, 32, 64)."""
    weights = []
    for layer_i in range(LAYERS):
        for i, (name, n, k, kind) in enumerate(PROJ):
            lat = synth.ternary_latents(n, k, seed=1000 + layer_i * 8 + i + 7000 * rank, device=dev)
            weights.append((a48.pack_ternary(lat, EPS, a48.LAYOUT_DECODE | a48.LAYOUT_SPARSE | a48.LAYOUT_GEMM), n, k, kind))
            del lat
    packed_bytes = sum(w.packed_bytes for w, *_ in weights)
    fused = not os.environ.get("A48_BENCH_DECODE_UNFUSED")

    def time_chain(M):
        x_h = synth.gaussian_outlier_activations(M, H, seed=50, device=dev)
        s_h = synth.student_t3(M, H, seed=51, device=dev)
        s_f = synth.student_t3(M, F, seed=52, device=dev)
        c4, d4 = a48.quant_int4(x_h, EPS)
        c8h, d8h, _ = a48.topk_quant_int8(s_h, H // 2, EPS)
        c8f, d8f, _ = a48.topk_quant_int8(s_f, F // 2, EPS)
        y = torch.empty(M, F, dtype=torch.float32, device=dev)
        ys = [torch.empty(M, F, dtype=torch.float32, device=dev) for _ in range(3)]
        yh = [torch.empty(M, H, dtype=torch.float32, device=dev) for _ in range(3)]
        ws_need = max(a48.linear_workspace_bytes(w, M) for w, *_ in weights[:7])
        ws_multi = max(a48.linear_multi_workspace_bytes([w for w, *_ in weights[0:3]], M),
                       a48.linear_multi_workspace_bytes([w for w, *_ in weights[4:6]], M), ws_need, 16)
        ws = torch.zeros(ws_multi, dtype=torch.uint8, device=dev)
        # channels with a non-zero code in at least one of the M tokens: the weight bytes a call really needs
        nz = {"int4": float((c4 != 0).any(0).float().mean()), "topk_h": float((c8h != 0).any(0).float().mean()),
              "topk_f": float((c8f != 0).any(0).float().mean())}
        needed_bytes = 0
        for w, n, k, kind in weights:
            needed_bytes += w.packed_bytes * (nz["int4"] if kind == "int4" else (nz["topk_h"] if k == H else nz["topk_f"]))

        def chain():
            # per layer: q,k,v share the attention input and gate,up the FFN input: one call each (one launch each)
            for li in range(LAYERS):
                (wq, *_), (wk, *_), (wv, *_), (wo, *_), (wg, *_), (wu, *_), (wd, *_) = weights[7 * li:7 * li + 7]
                if fused:
                    a48.linear_multi([wq, wk, wv], c4, d4, a48.ACT_INT4, Ys=yh, workspace=ws)
                else:
                    for w_, t in zip((wq, wk, wv), yh):
                        a48.linear(w_, c4, d4, a48.ACT_INT4, Y=t, workspace=ws)
                a48.linear(wo, c8h, d8h, a48.ACT_TOPK_INT8, Y=yh[0], workspace=ws)
                if fused:
                    a48.linear_multi([wg, wu], c4, d4, a48.ACT_INT4, Ys=[ys[0], ys[1]], workspace=ws)
                else:
                    a48.linear(wg, c4, d4, a48.ACT_INT4, Y=ys[0], workspace=ws)
                    a48.linear(wu, c4, d4, a48.ACT_INT4, Y=ys[1], workspace=ws)
                a48.linear(wd, c8f, d8f, a48.ACT_TOPK_INT8, Y=yh[0], workspace=ws)

        for _ in range(2):
            chain()
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            chain()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                chain()
        torch.cuda.synchronize()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 10
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        del graph
        return {"ms_all_bitlinears": ms, "weight_stream_gbs": packed_bytes / (ms * 1e-3) / 1e9,
                "algorithmic_gbs": needed_bytes / (ms * 1e-3) / 1e9, "tokens_per_s": M * 1e3 / ms,
                "dense_equivalent_tops": 2.0 * M * packed_bytes * 4 / (ms * 1e-3) / 1e12, "nonzero_channel_fraction": nz}

    by_tokens = {str(M): time_chain(M) for M in (1, 8, 32, 64)}
    one = by_tokens["1"]
    out = {"metric": "decode_weight_stream_gbs_7b_batch1", "value": one["weight_stream_gbs"], "unit": "GB/s",
           "ms_per_token_all_bitlinears": one["ms_all_bitlinears"], "packed_weight_bytes": packed_bytes,
           "matrices": len(weights), "hbm_peak_gbs": peaks["hbm_gbs"],
           "frac_of_hbm_peak": one["weight_stream_gbs"] / peaks["hbm_gbs"], "algorithmic_gbs": one["algorithmic_gbs"],
           "nonzero_code_fraction": one["nonzero_channel_fraction"], "tokens_per_s": one["tokens_per_s"],
           "launches_per_layer": 4 if fused else 7, "by_tokens": by_tokens,
           "note": "CUDA-graph chain over 224 distinct matrices (1.6 GB >> L2), q/k/v and gate/up each as one "
           "bitnet_a48_linear_multi call; value counts every packed byte, algorithmic_gbs only channels with a non-zero "
           "code in some token; 1 and 8 tokens run the streaming decode kernel, 32 and 64 the tensor-core kernel "
           "(64-token tile, cluster split-K)"}
    for w, *_ in weights:
        w.free()
    return out


def bench_block(a48, synth, dev, stream, layer):
    """Block forward tokens/s at the 7B shape: prefill 4096 x 4 and batch-1 decode at context 2048."""
    g1 = synth.norm_gains(H, 60, device=dev)
    g2 = synth.norm_gains(H, 61, device=dev)
    out = {}
    blk = a48.Block(layer.w, g1, g2, n_heads=NH, k_o=H // 2, k_down=F // 2, ctx_cap=4096)
    # prefill
    B, T = 4, 4096
    x = synth.gaussian_outlier_activations(B * T, H, seed=62, device=dev)
    ws = torch.empty(blk.workspace_bytes(B, T), dtype=torch.uint8, device=dev)
    y = torch.empty_like(x)
    kc = torch.zeros(B, NH, 4096, H // NH, dtype=torch.float32, device=dev)
    vc = torch.zeros_like(kc)
    blk.forward(x, B, T, 0, kc, vc, Y=y, workspace=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 2
    e0.record(stream)
    for _ in range(reps):
        blk.forward(x, B, T, 0, kc, vc, Y=y, workspace=ws)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    out["prefill"] = {"tokens_per_s": B * T / (ms * 1e-3), "ms": ms, "B": B, "T": T}
    # decode: one token per sequence against a 2048-token context
    for Bd in (1, 8):
        xd = synth.gaussian_outlier_activations(Bd, H, seed=63, device=dev)
        kcd = synth.kv_cache(Bd, NH, 4096, H // NH, seed=64, device=dev)
        vcd = synth.kv_cache(Bd, NH, 4096, H // NH, seed=65, device=dev)
        yd = torch.empty_like(xd)
        wsd = torch.empty(blk.workspace_bytes(Bd, 1), dtype=torch.uint8, device=dev)
        for _ in range(3):
            blk.forward(xd, Bd, 1, 2048, kcd, vcd, Y=yd, workspace=wsd)
        torch.cuda.synchronize()
        reps = 20
        e0.record(stream)
        for _ in range(reps):
            blk.forward(xd, Bd, 1, 2048, kcd, vcd, Y=yd, workspace=wsd)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        out[f"decode_b{Bd}"] = {"tokens_per_s": Bd / (ms * 1e-3), "ms": ms, "context": 2048}
        # the same call captured once in a CUDA graph (the call is stream-ordered, so a caller can do this)
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            blk.forward(xd, Bd, 1, 2048, kcd, vcd, Y=yd, workspace=wsd, stream=side)
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                blk.forward(xd, Bd, 1, 2048, kcd, vcd, Y=yd, workspace=wsd, stream=side)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        ms_g = e0.elapsed_time(e1) / reps
        out[f"decode_b{Bd}"].update({"ms_cuda_graph": ms_g, "tokens_per_s_cuda_graph": Bd / (ms_g * 1e-3)})
        del graph
    blk.free()
    out["note"] = "one 7B-shape block (fp32 attention glue included); tokens/s per block, not per model"
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-decode", action="store_true")
    ap.add_argument("--skip-block", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
