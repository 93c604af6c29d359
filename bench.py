#!/usr/bin/env python
"""Benchmark of the BitNet a4.8 BitLinear forward on B200.

One pass = the seven BitLinears of one 7B-shape transformer layer over 16384
tokens (prefill of 4096 tokens x batch 4): the per-token quantisers (INT4 for
the q/k/v and gate/up inputs, top-K 50 % + INT8 for the o and down inputs)
followed by the packed-ternary contractions and their rescale.  A counted step
is `passes_per_step` such passes, chosen so that the timed region lasts at
least a second whatever --steps says (the GPU then runs at the clock its power
cap leaves, not at a cold burst).  The headline value is dense-equivalent TOPS
(2*M*N*K summed over the seven projections, divided by the time of a pass,
quantisers included).  The same JSON line also carries the roofline of every
rated kernel, the end-to-end figure with host buffers, the CPU oracle timed on
a bounded sample, and one leg per remaining benchmark configuration: the decode
chains of the 7B and 3B shapes at 1/8/32/64 tokens, the 700M-shape prefill, the
M = 1..16384 sweep of the isolated BitLinear, and block tokens/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--legs a,b,...]

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

# DRAM bytes per launch of the prefill contraction (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture
# of the CTA-pair kernel at M = 4096, N = 11008, K = 4096: 150.9 MB against 208.5 MB of algorithmic bytes, part of
# the output still in L2 when the kernel ends), scaled by the units processed: x (488 MB / 208.5 MB), the mean
# algorithmic bytes M*K + N*K/4 + 4*M*N of the seven launches of a pass at M = 16384 over those of the captured case.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 150.9e6 * (488.0 / 208.5)
# DRAM bytes per launch of the quantisers from the ncu captures under profiles/ (read + write): top-K + INT8 at
# M = 4096, K = 11008 (180.5 + 28.1 MB) scaled x4 to 16384 tokens, traffic growing with the rows; INT4 at the
# benchmark's own shape (268.4 + 51.1 MB).  In both the input is read once; part of the output is still in L2 at kernel end.
NCU_TRAFFIC_TOPK_F = (180.5e6 + 28.1e6) * 4.0
NCU_TRAFFIC_INT4_H = 268.4e6 + 51.1e6
NOMINAL_INT8_TOPS = 4500.0  # dense int8 tensor peak of the part (2 x the 2.25 PFLOP/s dense bf16 figure)

# the other shapes of the paper's model-configuration table used by the legs
SHAPE_3B = dict(H=3200, F=8640, NH=32, LAYERS=26)
SHAPE_700M = dict(H=1536, F=4096, NH=16, LAYERS=24)  # 16 heads as the benchmark configuration fixes (head dim 96)
SHAPE_7B = dict(H=H, F=F, NH=NH, LAYERS=LAYERS)
ALL_LEGS = ("e2e", "decode7b", "decode3b", "prefill700m", "sweep", "block", "attention", "gatefirst", "formats", "cpu")


def proj_list(Hs, Fs):
    return (("q", Hs, Hs, "int4"), ("k", Hs, Hs, "int4"), ("v", Hs, Hs, "int4"), ("o", Hs, Hs, "topk"),
            ("gate", Fs, Hs, "int4"), ("up", Fs, Hs, "int4"), ("down", Hs, Fs, "topk"))


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
    """Packed weights of one transformer layer of a given shape."""

    def __init__(self, a48, dev, seed, layouts, Hs=H, Fs=F):
        from paper_2411_04965_b200 import synth
        self.w = {}
        for i, (name, n, k, _) in enumerate(proj_list(Hs, Fs)):
            lat = synth.ternary_latents(n, k, seed=seed * 16 + i, device=dev)
            self.w[name] = a48.pack_ternary(lat, EPS, layouts)
            del lat
        torch.cuda.synchronize()

    def free(self):
        for w in self.w.values():
            w.free()


class LayerStep:
    """The seven BitLinears of one layer on resident buffers: 4 quantiser launches and 7 contractions per pass."""

    KERNELS = ("int4_h", "q", "k", "v", "topk_h", "o", "int4_h2", "gate", "up", "topk_f", "down")

    def __init__(self, a48, synth, dev, layer, M, Hs, Fs, seed):
        self.a48, self.layer, self.M, self.H, self.F = a48, layer, M, Hs, Fs
        self.x_h = synth.gaussian_outlier_activations(M, Hs, seed=seed, device=dev)
        self.s_h = synth.student_t3(M, Hs, seed=seed + 1, device=dev)
        self.s_f = synth.student_t3(M, Fs, seed=seed + 2, device=dev)
        self.codes_h = torch.empty(M, Hs, dtype=torch.int8, device=dev)
        self.codes_f = torch.empty(M, Fs, dtype=torch.int8, device=dev)
        self.scale = torch.empty(M, dtype=torch.float32, device=dev)
        self.y_h = torch.empty(M, Hs, dtype=torch.float32, device=dev)
        self.y_f = torch.empty(M, Fs, dtype=torch.float32, device=dev)
        ws_need = max([a48.linear_workspace_bytes(w, M) for w in layer.w.values()] + [16])
        self.ws = torch.zeros(ws_need, dtype=torch.uint8, device=dev)
        self.ops = sum(2 * M * n * k for _, n, k, _ in proj_list(Hs, Fs))

    def run(self, stream, events=None):
        """One pass.  events: a list that receives one CUDA event before every launch and one after the last."""
        a48, w = self.a48, self.layer.w

        def mark():
            if events is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream)
                events.append(e)

        def lin(name, codes, kind, out):
            mark()
            a48.linear(w[name], codes, self.scale, kind, a48.ALGO_AUTO, Y=out, workspace=self.ws)

        mark()
        a48.quant_int4(self.x_h, EPS, self.codes_h, self.scale)
        for name in ("q", "k", "v"):
            lin(name, self.codes_h, a48.ACT_INT4, self.y_h)
        mark()
        a48.topk_quant_int8(self.s_h, self.H // 2, EPS, self.codes_h, self.scale)
        lin("o", self.codes_h, a48.ACT_TOPK_INT8, self.y_h)
        mark()
        a48.quant_int4(self.x_h, EPS, self.codes_h, self.scale)
        for name in ("gate", "up"):
            lin(name, self.codes_h, a48.ACT_INT4, self.y_f)
        mark()
        a48.topk_quant_int8(self.s_f, self.F // 2, EPS, self.codes_f, self.scale)
        lin("down", self.codes_f, a48.ACT_TOPK_INT8, self.y_h)
        mark()
        return len(self.KERNELS)  # kernel launches of this library per pass


def per_kernel_ms(pass_events):
    """Mean duration per kernel name over all passes: events sit before every launch and after the last."""
    sums = {}
    for ev in pass_events:
        for name, a, b in zip(LayerStep.KERNELS, ev[:-1], ev[1:]):
            sums.setdefault(name, []).append(a.elapsed_time(b))
    return {k: sum(v) / len(v) for k, v in sums.items()}


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
    legs = set(ALL_LEGS if args.legs == "all" else [l for l in args.legs.split(",") if l])
    unknown = legs - set(ALL_LEGS)
    if unknown:
        raise SystemExit(f"unknown legs {sorted(unknown)}; known: {ALL_LEGS}")
    if world > 1:  # the legs are single-GPU figures; every rank of a multi-GPU run would only repeat them
        legs &= {"e2e"}

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    max_over_ranks = reps.max_ms

    # ---- resident inputs: larger than L2 (268 MB + 268 MB + 721 MB of fp32 activations per pass)
    layer = Layer(a48, dev, seed=4 + rank, layouts=a48.LAYOUT_ALL)
    work = LayerStep(a48, synth, dev, layer, M, H, F, seed=40 + rank)

    sampler = ClockSampler(dev)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    work.run(stream)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(max(args.warmup, 3)):
        work.run(stream)
    e1.record(stream)
    barrier()
    est_ms = max_over_ranks(e0.elapsed_time(e1) / max(args.warmup, 3))
    # a counted step repeats the pass so that steps x passes x pass time >= the wanted length of the timed region
    passes = max(1, int(-(-args.min_region_ms // (args.steps * est_ms))))
    pass_events = []
    barrier()
    t_begin = time.time()
    e0.record(stream)
    launches = 0
    for _ in range(args.steps):
        for _ in range(passes):
            ev = []
            launches += work.run(stream, ev)
            pass_events.append(ev)
    e1.record(stream)
    barrier()
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end)
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    ms_per_step = ms_total / args.steps
    ms_per_pass = ms_per_step / passes
    tops = reps.job_value(STEP_OPS, ms_per_pass) / 1e12
    n_burst = min(20, len(pass_events))
    burst_ms = pass_events[0][0].elapsed_time(pass_events[n_burst - 1][-1]) / n_burst
    n_tail = max(1, len(pass_events) // 2)
    tail_ms = pass_events[-n_tail][0].elapsed_time(pass_events[-1][-1]) / n_tail

    kms = per_kernel_ms(pass_events)
    gemm_names = ("q", "k", "v", "o", "gate", "up", "down")
    gemm_ms = sum(kms[n] for n in gemm_names)
    gemm_ops = sum(2 * M * n * k for pn, n, k, _ in PROJ if pn in gemm_names)
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12
    # second denominator: nominal int8:bf16 ratio of 2 on the measured bf16 figure (sustained for a region >= 1 s)
    peak_kind = "bf16_tflops_sustained" if ms_total >= 1000.0 else "bf16_tflops"
    measured_x2 = 2.0 * peaks[peak_kind]
    roofline = {"bound": "tensor", "achieved": achieved, "peak": NOMINAL_INT8_TOPS, "unit": "TOPS",
                "frac": achieved / NOMINAL_INT8_TOPS, "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                "kernel": "BitLinear contraction (prefill, tcgen05 kind::i8 on CTA pairs)",
                "launches": 7 * len(pass_events), "avg_launch_ms": gemm_ms / 7,
                "peak_source": "nominal dense int8 tensor peak of the part (no int8 peak is measured on this pool)",
                "peak_measured_x2": measured_x2, "frac_of_measured": achieved / measured_x2,
                "peak_measured_source": f"2 x {peak_kind} of {peaks['source']} peaks (nominal int8:bf16 = 2)",
                "timed_region_ms": ms_total}
    lib = library_int8_tops(dev, stream) if rank == 0 else None
    if lib:
        roofline["library_int8_tops"] = lib
        roofline["library_int8_note"] = "torch._int_mm (vendor int8 GEMM) 8192^3, 20 calls, same GPU, outside the timed region"

    def hbm_entry(kernel, names, K, traffic=None):
        ms = sum(kms[n] for n in names) / len(names)
        bytes_ = 5.0 * M * K + 4.0 * M  # fp32 in, int8 out, one fp32 scale per token
        gbs = bytes_ / (ms * 1e-3) / 1e9
        return {"kernel": kernel, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "traffic": traffic, "avg_launch_ms": ms,
                "launches": len(names) * len(pass_events), "algorithmic_bytes_per_launch": bytes_,
                "peak_source": f"hbm_gbs of {peaks['source']} peaks"}

    rooflines = [dict(roofline),
                 hbm_entry("top-K + INT8 quantiser, 16384 x 11008 (Eq. 1, 3)", ("topk_f",), F, NCU_TRAFFIC_TOPK_F),
                 hbm_entry("top-K + INT8 quantiser, 16384 x 4096 (Eq. 1, 3)", ("topk_h",), H),
                 hbm_entry("INT4 quantiser, 16384 x 4096 (Eq. 7)", ("int4_h", "int4_h2"), H, NCU_TRAFFIC_INT4_H)]

    # ---- end to end with host buffers (pinned), copies inside the timed region
    e2e = bench_e2e(a48, dev, layer, work, reps, barrier, args) if "e2e" in legs else None
    del work
    torch.cuda.empty_cache()

    decode = decode3b = prefill700m = sweep = block = None
    if "decode7b" in legs:
        decode = bench_decode(a48, synth, dev, stream, peaks, rank, SHAPE_7B, "7b")
        one = decode["by_tokens"]["1"]
        rooflines.append({"kernel": "decode BitLinear chain, 7B shape, 1 token (224 matrices, CUDA graph)", "bound": "hbm",
                          "achieved": one["algorithmic_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": one["algorithmic_gbs"] / peaks["hbm_gbs"], "traffic": None,
                          "dense_gbs": one["weight_stream_gbs"],
                          "dense_frac": one["weight_stream_gbs"] / peaks["hbm_gbs"],
                          "note": "rated on algorithmic bytes (weight rows of channels with a non-zero code); "
                                  "dense_gbs counts every packed byte the kernel streams",
                          "peak_source": f"hbm_gbs of {peaks['source']} peaks"})
    if "decode3b" in legs:
        decode3b = bench_decode(a48, synth, dev, stream, peaks, rank, SHAPE_3B, "3b")
        decode3b["block"] = bench_block_decode(a48, synth, dev, stream, SHAPE_3B, (1, 8, 32, 64))
    if "prefill700m" in legs:
        prefill700m = bench_prefill_700m(a48, synth, dev, stream)
    if "sweep" in legs:
        sweep = bench_sweep(a48, synth, dev, stream)
    if "block" in legs:
        block = bench_block(a48, synth, dev, stream, layer)
    attention = None
    if "attention" in legs:
        attention = bench_attention(a48, synth, dev, stream, peaks)
        rooflines.append(attention.pop("roofline"))
    gate_first = bench_gate_first(a48, synth, dev, stream) if "gatefirst" in legs else None
    formats = None
    if "formats" in legs:
        formats = bench_formats(a48, synth, dev, stream, peaks, layer)
        rooflines.extend(formats.pop("rooflines"))

    cpu_baseline = None
    if rank == 0 and world == 1 and "cpu" in legs:
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
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x int2 -> int32 (scales fp64/fp32)", "data": "synthetic",
            "config": {"workload": "7B-shape layer (hidden 4096, GLU 11008): 7 BitLinears incl. quantisers, "
                                   "prefill 4096 tokens x batch 4 = 16384 tokens",
                       "passes_per_step": passes, "ms_per_pass": ms_per_pass,
                       "l2": "inputs larger than L2 (1.26 GB of fp32 activations + 1.3 GB of outputs per pass)",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "sustained": {"ms_per_pass": tail_ms, "tops": STEP_OPS / (tail_ms * 1e-3) / 1e12,
                          "window": f"last {n_tail} passes of the timed region"},
            "first_burst": {"ms_per_pass": burst_ms, "tops": STEP_OPS / (burst_ms * 1e-3) / 1e12,
                            "window": f"first {n_burst} passes of the timed region"},
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "rooflines": rooflines, "e2e": e2e,
            "cpu_baseline": cpu_baseline, "decode": decode, "decode_3b": decode3b, "prefill_700m": prefill700m,
            "sweep": sweep, "block": block, "attention": attention, "ffn_gate_first": gate_first, "formats": formats,
        }
        print(json.dumps(line))
    reps.close()


def bench_e2e(a48, dev, layer, work, reps, barrier, args):
    """The same pass through the host-buffer entry point: every call uploads its input and downloads its output."""
    M = work.M
    xh_host = work.x_h.cpu().pin_memory()
    sh_host = work.s_h.cpu().pin_memory()
    sf_host = work.s_f.cpu().pin_memory()
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
    dt = reps.max_ms((time.perf_counter() - t0) * 1e3) / n_e2e
    h2d = 6 * M * H * 4 + M * F * 4
    d2h = 5 * M * H * 4 + 2 * M * F * 4
    return {"value": STEP_OPS * reps.world / (dt * 1e-3) / 1e12, "unit": "TOPS", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": dt, "steps": n_e2e,
            "api": "bitnet_a48_bitlinear_host_async on 3 streams, pinned host buffers, stream sync per step"}


def graph_time_ms(fn, stream, reps, warm=3):
    """Captures fn() once in a CUDA graph on a side stream and returns the mean replay time."""
    fn()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            fn(side)
    torch.cuda.synchronize()
    for _ in range(warm):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    del graph
    return ms


def bench_decode(a48, synth, dev, stream, peaks, rank, shape, tag):
    """BitLinear chain over all 7 x LAYERS matrices of a model shape, one CUDA graph per token count (1, 8, 32, 64)."""
    Hs, Fs, layers = shape["H"], shape["F"], shape["LAYERS"]
    projs = proj_list(Hs, Fs)
    weights = []
    for layer_i in range(layers):
        for i, (name, n, k, kind) in enumerate(projs):
            lat = synth.ternary_latents(n, k, seed=1000 + layer_i * 8 + i + 7000 * rank, device=dev)
            weights.append((a48.pack_ternary(lat, EPS, a48.LAYOUT_DECODE | a48.LAYOUT_GEMM), n, k, kind))
            del lat
    packed_bytes = sum(w.packed_bytes for w, *_ in weights)

    def time_chain(M):
        x_h = synth.gaussian_outlier_activations(M, Hs, seed=50, device=dev)
        s_h = synth.student_t3(M, Hs, seed=51, device=dev)
        s_f = synth.student_t3(M, Fs, seed=52, device=dev)
        c4, d4 = a48.quant_int4(x_h, EPS)
        c8h, d8h, _ = a48.topk_quant_int8(s_h, Hs // 2, EPS)
        c8f, d8f, _ = a48.topk_quant_int8(s_f, Fs // 2, EPS)
        ys = [torch.empty(M, Fs, dtype=torch.float32, device=dev) for _ in range(2)]
        yh = [torch.empty(M, Hs, dtype=torch.float32, device=dev) for _ in range(3)]
        ws_need = max(a48.linear_workspace_bytes(w, M) for w, *_ in weights[:7])
        ws_multi = max(a48.linear_multi_workspace_bytes([w for w, *_ in weights[0:3]], M),
                       a48.linear_multi_workspace_bytes([w for w, *_ in weights[4:6]], M), ws_need, 16)
        ws = torch.zeros(ws_multi, dtype=torch.uint8, device=dev)
        # channels with a non-zero code in at least one of the M tokens: the weight bytes a call really needs
        nz = {"int4": float((c4 != 0).any(0).float().mean()), "topk_h": float((c8h != 0).any(0).float().mean()),
              "topk_f": float((c8f != 0).any(0).float().mean())}
        needed_bytes = 0
        for w, n, k, kind in weights:
            needed_bytes += w.packed_bytes * (nz["int4"] if kind == "int4" else (nz["topk_h"] if k == Hs else nz["topk_f"]))

        def chain(st=None):
            # per layer: q,k,v share the attention input and gate,up the FFN input: one call each (one launch each)
            for li in range(layers):
                (wq, *_), (wk, *_), (wv, *_), (wo, *_), (wg, *_), (wu, *_), (wd, *_) = weights[7 * li:7 * li + 7]
                a48.linear_multi([wq, wk, wv], c4, d4, a48.ACT_INT4, Ys=yh, workspace=ws, stream=st)
                a48.linear(wo, c8h, d8h, a48.ACT_TOPK_INT8, Y=yh[0], workspace=ws, stream=st)
                a48.linear_multi([wg, wu], c4, d4, a48.ACT_INT4, Ys=ys, workspace=ws, stream=st)
                a48.linear(wd, c8f, d8f, a48.ACT_TOPK_INT8, Y=yh[0], workspace=ws, stream=st)

        chain()
        ms = graph_time_ms(chain, stream, reps=10)
        return {"ms_all_bitlinears": ms, "weight_stream_gbs": packed_bytes / (ms * 1e-3) / 1e9,
                "algorithmic_gbs": needed_bytes / (ms * 1e-3) / 1e9, "tokens_per_s": M * 1e3 / ms,
                "dense_equivalent_tops": 2.0 * M * packed_bytes * 4 / (ms * 1e-3) / 1e12, "nonzero_channel_fraction": nz}

    by_tokens = {str(M): time_chain(M) for M in (1, 8, 32, 64)}
    one = by_tokens["1"]
    out = {"metric": f"decode_weight_stream_gbs_{tag}_batch1", "value": one["weight_stream_gbs"], "unit": "GB/s",
           "ms_per_token_all_bitlinears": one["ms_all_bitlinears"], "packed_weight_bytes": packed_bytes,
           "matrices": len(weights), "hbm_peak_gbs": peaks["hbm_gbs"],
           "frac_of_hbm_peak": one["weight_stream_gbs"] / peaks["hbm_gbs"], "algorithmic_gbs": one["algorithmic_gbs"],
           "algorithmic_frac_of_hbm_peak": one["algorithmic_gbs"] / peaks["hbm_gbs"],
           "nonzero_code_fraction": one["nonzero_channel_fraction"], "tokens_per_s": one["tokens_per_s"],
           "launches_per_layer": 4, "by_tokens": by_tokens,
           "note": f"CUDA-graph chain over {len(weights)} distinct matrices ({packed_bytes / 1e9:.2f} GB >> L2), q/k/v and "
           "gate/up each as one bitnet_a48_linear_multi call; value counts every packed byte, algorithmic_gbs only "
           "channels with a non-zero code in some token; 1 and 8 tokens run the streaming decode kernel, 32 and 64 the "
           "tensor-core kernel (64-token tile, cluster split-K)"}
    for w, *_ in weights:
        w.free()
    return out


def bench_block_decode(a48, synth, dev, stream, shape, batches, ctx=2048, layer=None, q_bits=0, kv_bits=0):
    """One block forward per new token against a context of `ctx` cached positions, per batch size.

    kv_bits != 0: the packed low-bit cache, filled by a prefill of `ctx` tokens through the block itself."""
    Hs, Fs, nh = shape["H"], shape["F"], shape["NH"]
    own = layer is None
    if own:
        layer = Layer(a48, dev, seed=77, layouts=a48.LAYOUT_ALL, Hs=Hs, Fs=Fs)
    g1 = synth.norm_gains(Hs, 60, device=dev)
    g2 = synth.norm_gains(Hs, 61, device=dev)
    cap = ctx + 8
    blk = a48.Block(layer.w, g1, g2, n_heads=nh, k_o=Hs // 2, k_down=Fs // 2, ctx_cap=cap, q_bits=q_bits, kv_bits=kv_bits)
    out = {}
    for Bd in batches:
        xd = synth.gaussian_outlier_activations(Bd, Hs, seed=63, device=dev)
        if kv_bits:
            kcd = torch.zeros(blk.kv_cache_bytes(Bd), dtype=torch.uint8, device=dev)
            vcd = torch.zeros_like(kcd)
            xp = synth.gaussian_outlier_activations(Bd * ctx, Hs, seed=66, device=dev)
            blk.forward(xp, Bd, ctx, 0, kcd, vcd)
            torch.cuda.synchronize()
            del xp
            torch.cuda.empty_cache()
        else:
            kcd = synth.kv_cache(Bd, nh, cap, Hs // nh, seed=64, device=dev)
            vcd = synth.kv_cache(Bd, nh, cap, Hs // nh, seed=65, device=dev)
        yd = torch.empty_like(xd)
        wsd = torch.empty(blk.workspace_bytes(Bd, 1), dtype=torch.uint8, device=dev)

        def call(st=None):
            blk.forward(xd, Bd, 1, ctx, kcd, vcd, Y=yd, workspace=wsd, stream=st)

        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        e0.record(stream)
        for _ in range(reps):
            call()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        ms_g = graph_time_ms(call, stream, reps=reps)  # the call is stream-ordered, so a caller can capture it
        out[f"b{Bd}"] = {"tokens_per_s": Bd / (ms * 1e-3), "ms": ms, "context": ctx, "ms_cuda_graph": ms_g,
                         "tokens_per_s_cuda_graph": Bd / (ms_g * 1e-3),
                         "kv_cache_bytes": 2 * (kcd.numel() * kcd.element_size())}
        del kcd, vcd
    blk.free()
    if own:
        layer.free()
    return out


def bench_prefill_700m(a48, synth, dev, stream):
    """700M shape: the seven BitLinears of a layer and the whole block on a 2048-token prefill at batch 1."""
    Hs, Fs, nh, layers = SHAPE_700M["H"], SHAPE_700M["F"], SHAPE_700M["NH"], SHAPE_700M["LAYERS"]
    T = 2048
    layer = Layer(a48, dev, seed=88, layouts=a48.LAYOUT_ALL, Hs=Hs, Fs=Fs)
    work = LayerStep(a48, synth, dev, layer, T, Hs, Fs, seed=90)
    ms = graph_time_ms(lambda st=None: work.run(st if st is not None else stream), stream, reps=50)
    out = {"bitlinears_ms_per_layer": ms, "bitlinears_tops": work.ops / (ms * 1e-3) / 1e12,
           "bitlinears_tokens_per_s_model": T / (ms * 1e-3 * layers)}
    g1 = synth.norm_gains(Hs, 60, device=dev)
    g2 = synth.norm_gains(Hs, 61, device=dev)
    blk = a48.Block(layer.w, g1, g2, n_heads=nh, k_o=Hs // 2, k_down=Fs // 2, ctx_cap=0)
    x = synth.gaussian_outlier_activations(T, Hs, seed=62, device=dev)
    y = torch.empty_like(x)
    ws = torch.empty(blk.workspace_bytes(1, T), dtype=torch.uint8, device=dev)
    ms_b = graph_time_ms(lambda st=None: blk.forward(x, 1, T, 0, None, None, Y=y, workspace=ws, stream=st), stream, reps=20)
    out.update({"block_ms": ms_b, "block_tokens_per_s": T / (ms_b * 1e-3),
                "model_tokens_per_s": T / (ms_b * 1e-3 * layers),
                "note": "hidden 1536, GLU 4096, 16 heads of 96, 2048 tokens, batch 1; per-layer figures, the model figure "
                        "divides by 24 layers (no embedding or head)"})
    blk.free()
    layer.free()
    return out


def bench_sweep(a48, synth, dev, stream, copies=12, reps=5):
    """Isolated BitLinear (the library's own choice of kernel) for M = 1, 2, 4, .., 16384 on the two 7B feed-forward
    shapes with INT4 and top-K codes: one CUDA graph per point over `copies` distinct matrices, so that neither the
    host's launch cost nor L2 residency of the weights enters the figure."""
    points = []
    for N, K in ((F, H), (H, F)):
        ws = [a48.pack_ternary(synth.ternary_latents(N, K, seed=100 + i, device=dev), EPS,
                               a48.LAYOUT_DECODE | a48.LAYOUT_GEMM) for i in range(copies)]
        for kind in ("int4", "topk"):
            for e in range(15):
                M = 1 << e
                if kind == "int4":
                    codes, scale = a48.quant_int4(synth.gaussian_outlier_activations(M, K, seed=11, device=dev), EPS)
                    act = a48.ACT_INT4
                else:
                    codes, scale, _ = a48.topk_quant_int8(synth.student_t3(M, K, seed=12, device=dev), K // 2, EPS)
                    act = a48.ACT_TOPK_INT8
                y = torch.empty(M, N, dtype=torch.float32, device=dev)
                wsp = torch.zeros(max(a48.linear_workspace_bytes(ws[0], M), 16), dtype=torch.uint8, device=dev)
                use = ws if M <= 1024 else ws[:2]  # large M: the activations alone exceed L2

                def run(st=None):
                    for w in use:
                        a48.linear(w, codes, scale, act, Y=y, workspace=wsp, stream=st)

                ms = graph_time_ms(run, stream, reps=reps, warm=1) / len(use)
                points.append({"N": N, "K": K, "kind": kind, "M": M, "us": ms * 1e3,
                               "dense_tops": 2.0 * M * N * K / ms / 1e9, "weight_gbs": ws[0].packed_bytes / ms / 1e6})
                del y, codes
        for w in ws:
            w.free()
    return {"points": points,
            "note": "bitnet_a48_linear alone (codes resident), time per call; dense_tops = 2*M*N*K / time, weight_gbs = "
                    "packed weight bytes / time"}


def time_ms(fn, stream, reps, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def bench_attention(a48, synth, dev, stream, peaks):
    """Prefill attention of the 7B shape on its own: 4 sequences of 4096 tokens, 32 heads of 128 (the block leg's shape)."""
    B, T, nh, hd = 4, 4096, NH, H // NH
    g = torch.Generator(device=dev).manual_seed(91)
    q = torch.randn(B * T, nh * hd, generator=g, device=dev)
    kc = synth.kv_cache(B, nh, T, hd, seed=92, device=dev)
    vc = synth.kv_cache(B, nh, T, hd, seed=93, device=dev)
    out = torch.empty_like(q)
    ws = torch.empty(a48.attention_prefill_workspace_bytes(B, nh, hd, T, T), dtype=torch.uint8, device=dev)
    ms = time_ms(lambda: a48.attention_prefill(q, kc, vc, B, T, 0, out=out, workspace=ws), stream, 10)
    flops = 4.0 * B * nh * (T * (T + 1) / 2.0) * hd  # q.k and p.v for every visible (query, key) pair
    tiles = B * nh * sum(min(2 * (i + 1), T // 64) for i in range(T // 128))  # key tiles of 64 per 128-query tile
    mma_flops = tiles * 6.0 * 2 * (2.0 * 128 * 64 * hd)  # six bf16 MMAs per product, whole tiles, both contractions
    tf = flops / (ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    roof = {"kernel": "prefill attention, 4 x 4096 tokens, 32 heads of 128 (tcgen05 kind::f16 on bf16-split operands; "
                      "three launches that split the operands included)",
            "bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak, "traffic": None,
            "avg_launch_ms": ms, "algorithmic_flops_per_launch": flops,
            "mma_tflops": mma_flops / (ms * 1e-3) / 1e12, "mma_frac": mma_flops / (ms * 1e-3) / 1e12 / peak,
            "note": "achieved counts the attention's own flops; the kernel issues six bf16 MMAs per fp32 product to stay "
                    "within fp32 rounding of the float64 oracle (mma_tflops counts those, whole tiles)",
            "peak_source": f"bf16_tflops of {peaks['source']} peaks"}
    del q, kc, vc, out, ws
    torch.cuda.empty_cache()
    return {"ms": ms, "tokens_per_s": B * T / (ms * 1e-3), "B": B, "T": T, "heads": nh, "head_dim": hd, "roofline": roof}


def bench_formats(a48, synth, dev, stream, peaks, layer):
    """The other number formats of the library on the 7B shape: FP4 quantiser (Eq. 8-9), bf16 activations at the
    boundary, and the five-codes-per-byte weight layout in a decode chain."""
    M = M_PREFILL
    out, roof = {}, []

    def hbm(kernel, ms, bytes_):
        gbs = bytes_ / (ms * 1e-3) / 1e9
        return {"kernel": kernel, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "traffic": None, "avg_launch_ms": ms,
                "algorithmic_bytes_per_launch": bytes_, "peak_source": f"hbm_gbs of {peaks['source']} peaks"}

    x = synth.gaussian_outlier_activations(M, H, seed=45, device=dev)
    codes = torch.empty(M, H, dtype=torch.int8, device=dev)
    scale = torch.empty(M, dtype=torch.float32, device=dev)
    ms = time_ms(lambda: a48.quant_fp4(x, codes, scale), stream, 50)
    roof.append(hbm("FP4 (E2M1) quantiser, 16384 x 4096 (Eq. 8-9)", ms, 5.0 * M * H + 4.0 * M))
    # bf16 in, bf16 out: INT4 quantiser and the gate projection
    xb = x.to(torch.bfloat16)
    ms = time_ms(lambda: a48.quant_int4_bf16(xb, EPS, codes, scale), stream, 50)
    roof.append(hbm("INT4 quantiser from bf16 rows, 16384 x 4096 (Eq. 7)", ms, 3.0 * M * H + 4.0 * M))
    sb = synth.student_t3(M, F, seed=46, device=dev).to(torch.bfloat16)
    codes_f = torch.empty(M, F, dtype=torch.int8, device=dev)
    ms = time_ms(lambda: a48.topk_quant_int8_bf16(sb, F // 2, EPS, codes_f, scale), stream, 20)
    roof.append(hbm("top-K + INT8 quantiser from bf16 rows, 16384 x 11008 (Eq. 1, 3)", ms, 3.0 * M * F + 4.0 * M))
    del sb, codes_f
    a48.quant_int4(x, EPS, codes, scale)
    y32 = torch.empty(M, F, dtype=torch.float32, device=dev)
    y16 = torch.empty(M, F, dtype=torch.bfloat16, device=dev)
    ops = 2.0 * M * F * H
    ms32 = time_ms(lambda: a48.linear(layer.w["gate"], codes, scale, a48.ACT_INT4, Y=y32), stream, 100)
    ms16 = time_ms(lambda: a48.linear_bf16(layer.w["gate"], codes, scale, a48.ACT_INT4, Y=y16), stream, 100)
    out["gate_projection_16384_tokens"] = {"fp32_out_ms": ms32, "fp32_out_tops": ops / ms32 / 1e9, "bf16_out_ms": ms16,
                                           "bf16_out_tops": ops / ms16 / 1e9,
                                           "note": "bitnet_a48_linear against bitnet_a48_linear_bf16, 100 calls each"}
    del y32, y16, x, xb
    torch.cuda.empty_cache()
    # five codes per byte: the seven matrices of 16 distinct layers in one CUDA graph (0.65 GB >> L2), 1 and 8 tokens
    layers = 16
    ws5, ws2 = [], []
    for li in range(layers):
        for i, (name, n, k, kind) in enumerate(PROJ):
            lat = synth.ternary_latents(n, k, seed=5000 + li * 8 + i, device=dev)
            w = a48.pack_ternary(lat, EPS, a48.LAYOUT_TRIT5 | a48.LAYOUT_DECODE)
            ws5.append((w, n, k, kind))
            del lat
    b5 = sum(w.layout_bytes(a48.LAYOUT_TRIT5) for w, *_ in ws5)
    b2 = sum(w.packed_bytes for w, *_ in ws5)
    out["trit5"] = {"bytes_five_per_byte": b5, "bytes_two_bit": b2, "ratio": b5 / b2, "layers": layers}
    for Mt in (1, 8):
        c4, d4 = a48.quant_int4(synth.gaussian_outlier_activations(Mt, H, seed=50, device=dev), EPS)
        c8h, d8h, _ = a48.topk_quant_int8(synth.student_t3(Mt, H, seed=51, device=dev), H // 2, EPS)
        c8f, d8f, _ = a48.topk_quant_int8(synth.student_t3(Mt, F, seed=52, device=dev), F // 2, EPS)
        yh = torch.empty(Mt, H, dtype=torch.float32, device=dev)
        yf = torch.empty(Mt, F, dtype=torch.float32, device=dev)
        wsp = torch.zeros(max(a48.linear_workspace_bytes(w, Mt) for w, *_ in ws5[:7]), dtype=torch.uint8, device=dev)

        def chain(algo, st=None):
            for w, n, k, kind in ws5:
                c, d, act = (c4, d4, a48.ACT_INT4) if kind == "int4" else ((c8h, d8h, a48.ACT_TOPK_INT8) if k == H else (c8f, d8f, a48.ACT_TOPK_INT8))
                a48.linear(w, c, d, act, algo, Y=yf if n == F else yh, workspace=wsp, stream=st)

        ms5 = graph_time_ms(lambda st=None: chain(a48.ALGO_DECODE_TRIT5, st), stream, reps=10)
        ms2 = graph_time_ms(lambda st=None: chain(a48.ALGO_DECODE, st), stream, reps=10)
        out["trit5"][f"tokens_{Mt}"] = {"five_per_byte_ms": ms5, "five_per_byte_gbs": b5 / ms5 / 1e6, "two_bit_ms": ms2,
                                        "two_bit_gbs": b2 / ms2 / 1e6,
                                        "note": "one launch per matrix in both chains (no fused q/k/v, gate/up launches)"}
    for w, *_ in ws5:
        w.free()
    out["rooflines"] = roof
    return out


def bench_gate_first(a48, synth, dev, stream, layers=16):
    """Feed-forward sub-layer of the 7B shape for 1 and 4 tokens, dense against gate-first, over `layers` distinct
    layers in one CUDA graph (0.54 GB of packed weights, larger than L2)."""
    ws_ = []
    for li in range(layers):
        trip = []
        for i, (n, k) in enumerate(((F, H), (F, H), (H, F))):
            lat = synth.latent_weights(n, k, seed=3000 + li * 4 + i, device=dev)
            trip.append(a48.pack_ternary(lat, EPS, a48.LAYOUT_DECODE))
            del lat
        ws_.append(trip)
    dense_bytes = sum(w.packed_bytes for w in ws_[0])
    out = {"dense_weight_bytes_per_layer": dense_bytes, "layers": layers}
    for M in (1, 4):
        x = synth.gaussian_outlier_activations(M, H, seed=70, device=dev)
        y = torch.empty(M, H, dtype=torch.float32, device=dev)
        work = torch.empty(a48.ffn_workspace_bytes(*ws_[0], M), dtype=torch.uint8, device=dev)
        _, _, rows = a48.ffn_gate_first(*ws_[0], x, F // 2, EPS, want_rows=True)
        torch.cuda.synchronize()
        rows_fetched = int(rows[0])

        def dense(st=None):
            for g, u, d in ws_:
                a48.ffn_dense(g, u, d, x, F // 2, EPS, Y=y, workspace=work, stream=st)

        def gate_first(st=None):
            for g, u, d in ws_:
                a48.ffn_gate_first(g, u, d, x, F // 2, EPS, Y=y, workspace=work, stream=st)

        ms_d = graph_time_ms(dense, stream, reps=10) / layers
        ms_g = graph_time_ms(gate_first, stream, reps=10) / layers
        up_bytes = ws_[0][1].packed_bytes
        fetched = dense_bytes - up_bytes + up_bytes * rows_fetched / F
        out[f"tokens_{M}"] = {"dense_us": ms_d * 1e3, "gate_first_us": ms_g * 1e3, "up_rows_fetched": rows_fetched,
                              "up_rows_fetched_fraction": rows_fetched / F, "weight_bytes_fetched": fetched,
                              "weight_bytes_fetched_fraction": fetched / dense_bytes,
                              "dense_gbs": dense_bytes / ms_d / 1e6, "gate_first_algorithmic_gbs": fetched / ms_g / 1e6}
    for trip in ws_:
        for w in trip:
            w.free()
    out["note"] = ("bitnet_a48_ffn_dense against bitnet_a48_ffn_gate_first: INT4 quantiser, gate/up, Eq. 5, top-K + INT8, "
                   "down; synthetic Gaussian latents give about half positive gates (the paper reports 67.5 % zero gates "
                   "on trained 7B weights)")
    return out


def bench_block(a48, synth, dev, stream, layer):
    """Block forward tokens/s at the 7B shape: prefill 4096 x 4 and decode at context 2048."""
    g1 = synth.norm_gains(H, 60, device=dev)
    g2 = synth.norm_gains(H, 61, device=dev)
    out = {}
    blk = a48.Block(layer.w, g1, g2, n_heads=NH, k_o=H // 2, k_down=F // 2, ctx_cap=4096)
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
    blk.free()
    del x, y, ws, kc, vc
    torch.cuda.empty_cache()
    dec = bench_block_decode(a48, synth, dev, stream, SHAPE_7B, (1, 8), layer=layer)
    out["decode_b1"], out["decode_b8"] = dec["b1"], dec["b8"]
    # the same steps with 4-bit queries and a 3-bit key/value cache (Section 3, low-bit attention)
    low = bench_block_decode(a48, synth, dev, stream, SHAPE_7B, (1, 8), layer=layer, q_bits=4, kv_bits=3)
    out["decode_b1_q4_kv3"], out["decode_b8_q4_kv3"] = low["b1"], low["b8"]
    out["note"] = "one 7B-shape block, attention included (prefill: tcgen05 on bf16-split operands; decode: fp32 or packed low-bit cache); tokens/s per block, not per model"
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--legs", default="all",
                    help="comma-separated extra legs beside the main step (" + ",".join(ALL_LEGS) + "), 'all' or ''")
    ap.add_argument("--min-region-ms", type=float, default=1000.0,
                    help="the timed region lasts at least this long: a counted step repeats the pass as often as needed")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
