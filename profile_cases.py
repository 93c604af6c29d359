"""Small single-kernel cases for profiler captures (ncu) and quick timing.

    python profile_cases.py gemm   --M 8192 --N 11008 --K 4096 --kind int4 --reps 3
    python profile_cases.py quant  --M 16384 --K 4096 --kind topk --reps 3
    python profile_cases.py decode --M 1 --N 11008 --K 4096 --kind topk --copies 32 --reps 3
    python profile_cases.py block  --B 1 --T 2048 --hidden 4096 --ffn 11008 --heads 32 --reps 3
    python profile_cases.py block  --B 1 --T 1 --ctx 2048 --reps 4          # one decode step against a cached context

Each case builds seeded synthetic inputs (the same recipes the benchmark uses),
runs the kernel `reps` times after one warm-up call and prints the mean time
from CUDA events on the launching stream.  `decode` cycles over `copies`
distinct weight matrices so that the weight bytes come from HBM, not L2.  `block` is one transformer block on a
prefill of B sequences of T tokens (quantisers, the seven BitLinears, RoPE, the tensor-core attention).
(The sweep over the token count is a leg of the benchmark: `python bench.py --legs sweep`.)
"""
from __future__ import annotations

import argparse
import json

import torch

from paper_2411_04965_b200 import binding as a48
from paper_2411_04965_b200 import build as a48_build
from paper_2411_04965_b200 import synth

EPS = 1e-5


def _time(fn, reps, stream):
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def _acts(kind, M, K, dev, k_frac=0.5):
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed=11, device=dev)
        codes, scale = a48.quant_int4(x, EPS)
        return x, codes, scale, a48.ACT_INT4
    x = synth.student_t3(M, K, seed=12, device=dev)
    codes, scale, _ = a48.topk_quant_int8(x, max(1, int(K * k_frac)), EPS)
    return x, codes, scale, a48.ACT_TOPK_INT8


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["gemm", "quant", "decode", "block"])
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--N", type=int, default=11008)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--kind", choices=["int4", "topk", "fp4"], default="int4")
    ap.add_argument("--algo", type=int, default=a48.ALGO_AUTO)
    ap.add_argument("--copies", type=int, default=32)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--B", type=int, default=1)
    ap.add_argument("--T", type=int, default=2048)
    ap.add_argument("--hidden", type=int, default=4096)
    ap.add_argument("--ffn", type=int, default=11008)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--ctx", type=int, default=0, help="block: cached positions in front of the call (fp32 cache), e.g. a decode step")
    args = ap.parse_args()
    a48_build.build()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    stream = torch.cuda.current_stream()
    M, N, K = args.M, args.N, args.K
    out = {"case": args.case, "M": M, "N": N, "K": K, "kind": args.kind}
    if args.case == "block":
        Hs, Fs, B, T = args.hidden, args.ffn, args.B, args.T
        shapes = (("q", Hs, Hs), ("k", Hs, Hs), ("v", Hs, Hs), ("o", Hs, Hs), ("gate", Fs, Hs), ("up", Fs, Hs), ("down", Hs, Fs))
        w = {n: a48.pack_ternary(synth.ternary_latents(r, c, seed=200 + i, device=dev), EPS, a48.LAYOUT_ALL)
             for i, (n, r, c) in enumerate(shapes)}
        blk = a48.Block(w, synth.norm_gains(Hs, 60, device=dev), synth.norm_gains(Hs, 61, device=dev), n_heads=args.heads,
                        k_o=Hs // 2, k_down=Fs // 2, ctx_cap=args.ctx + T if args.ctx > 0 else 0)
        x = synth.gaussian_outlier_activations(B * T, Hs, seed=13, device=dev)
        y = torch.empty_like(x)
        wsp = torch.empty(blk.workspace_bytes(B, T), dtype=torch.uint8, device=dev)
        if args.ctx > 0:
            kc = synth.kv_cache(B, args.heads, args.ctx + T, Hs // args.heads, seed=14, device=dev)
            vc = synth.kv_cache(B, args.heads, args.ctx + T, Hs // args.heads, seed=15, device=dev)
            ms = _time(lambda: blk.forward(x, B, T, args.ctx, kc, vc, Y=y, workspace=wsp), args.reps, stream)
        else:
            ms = _time(lambda: blk.forward(x, B, T, Y=y, workspace=wsp), args.reps, stream)
        hd = Hs // args.heads
        out = {"case": "block", "B": B, "T": T, "hidden": Hs, "ffn": Fs, "heads": args.heads, "ms": ms,
               "tokens_per_s": B * T / (ms * 1e-3), "attention_gflop": 4.0 * B * args.heads * (T * T / 2.0) * hd / 1e9}
    elif args.case == "quant":
        x = (synth.student_t3 if args.kind == "topk" else synth.gaussian_outlier_activations)(M, K, 11, device=dev)
        codes = torch.empty(M, K, dtype=torch.int8, device=dev)
        scale = torch.empty(M, dtype=torch.float32, device=dev)
        if args.kind == "int4":
            ms = _time(lambda: a48.quant_int4(x, EPS, codes, scale), args.reps, stream)
        elif args.kind == "fp4":
            ms = _time(lambda: a48.quant_fp4(x, codes, scale), args.reps, stream)
        else:
            ms = _time(lambda: a48.topk_quant_int8(x, K // 2, EPS, codes, scale), args.reps, stream)
        out.update(ms=ms, gbs=(5.0 * M * K + 4 * M) / ms / 1e6)
    elif args.case == "gemm":
        algo = args.algo or (a48.ALGO_GEMM_TCGEN05_PAIR if M >= 1024 else a48.ALGO_GEMM_TCGEN05)
        layouts = a48.LAYOUT_GEMM | (a48.LAYOUT_I8 if algo == a48.ALGO_GEMM_TCGEN05_I8 else 0)
        w = a48.pack_ternary(synth.ternary_latents(N, K, seed=4, device=dev), EPS, layouts)
        _, codes, scale, act = _acts(args.kind, M, K, dev)
        y = torch.empty(M, N, dtype=torch.float32, device=dev)
        ms = _time(lambda: a48.linear(w, codes, scale, act, algo, Y=y), args.reps, stream)
        out.update(ms=ms, tops=2.0 * M * N * K / ms / 1e9)
    else:
        ws = [a48.pack_ternary(synth.ternary_latents(N, K, seed=100 + i, device=dev), EPS,
                               a48.LAYOUT_DECODE | a48.LAYOUT_SPARSE) for i in range(args.copies)]
        _, codes, scale, act = _acts(args.kind, M, K, dev)
        y = torch.empty(M, N, dtype=torch.float32, device=dev)
        need = a48.linear_workspace_bytes(ws[0], M)
        wsp = torch.zeros(max(need, 16), dtype=torch.uint8, device=dev)

        def run():
            for w in ws:
                a48.linear(w, codes, scale, act, args.algo, Y=y, workspace=wsp)

        ms = _time(run, args.reps, stream) / len(ws)
        out.update(ms=ms, dense_gbs=ws[0].packed_bytes / ms / 1e6)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
