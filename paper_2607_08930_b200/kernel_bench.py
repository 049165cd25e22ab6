"""Per-kernel timings through the single-operation entry points (CUDA events, L2 flushed between launches).

    python -m paper_2607_08930_b200.kernel_bench gemm --shape dream --m 32 256 2048
    python -m paper_2607_08930_b200.kernel_bench attention --shape llada --rows 48 --vis 600
    python -m paper_2607_08930_b200.kernel_bench confidence --rows 512 --vocab 152064

Prints one line per case: microseconds (median of `--iters`), algorithmic TFLOP/s and GB/s.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as B

SHAPES = {   # d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab
    "dream": (3584, 28, 4, 128, 18944, 152064),
    "llada": (4096, 32, 32, 128, 12288, 126464),
    "tiny": (256, 4, 4, 64, 704, 1024),
}


def _time_graph(run, reps, iters):
    """Average device time of one launch: `reps` launches are captured into a CUDA graph and replayed, so the
    measurement does not depend on how fast the host can issue them."""
    for i in range(3):
        run(i)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(reps):
                run(i)
    ts = []
    for _ in range(iters + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) / reps)
    return float(np.median(ts[1:])) * 1e-3


def _time(fn, iters, flush):
    for _ in range(3):
        fn()
    ts = []
    for _ in range(iters):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return float(np.median(ts)) * 1e-3


def bench_gemm(args):
    """Back-to-back launches over rotating weight copies (together larger than L2, so every launch streams its
    weights from HBM); the reported time is the average per launch, free of launch-gap artefacts."""
    d, hq, hkv, dh, ffn, vocab = SHAPES[args.shape]
    gemms = {"qkv": ((hq + 2 * hkv) * dh, d, 0), "o": (d, hq * dh, 1), "gate_up": (ffn, d, 3), "down": (d, ffn, 1),
             "lm_head": (vocab, d, 2), "lm_head_conf": (vocab, d, 5)}
    scratch = torch.empty(16 << 20, dtype=torch.float32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    for name, (N, K, mode) in gemms.items():
        if args.only and name not in args.only:
            continue
        nw = 2 if mode == 3 else 1
        copies = 1 if args.hot else max(2, -(-(320 << 20) // (N * K * 2 * nw)))
        Ws = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(copies)]
        W2s = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(copies)] if mode == 3 else None
        for M in args.m:
            if name.startswith("lm_head") and M > 2048:
                continue
            A = torch.randn(M, K, device="cuda").bfloat16()
            rs = torch.ones(M, device="cuda") if mode in (2, 5) else None
            if mode == 5:      # the LM head with the confidence pass in its epilogue (GEMM + slice merge + final merge)
                bufs = B.lm_head_confidence_buffers(M, N, "cuda")
                flag = bufs["flag"]

                def run(i):
                    B.op_lm_head_confidence(A, Ws[i % copies], rs, N - 1, buffers=bufs)

                out_bytes = 2.0 * 12.0 * M * ((N + 31) // 32)       # group partials written, then read once
            else:
                Cd = torch.zeros(M, N, device="cuda", dtype=torch.bfloat16 if mode in (0, 3) else torch.float32)

                def run(i):
                    B.op_gemm(A, Ws[i % copies], mode, W2=None if W2s is None else W2s[i % copies], C_out=Cd,
                              row_scale=rs, scratch=scratch, error_flag=flag)

                out_bytes = Cd.numel() * Cd.element_size() * (2 if mode == 1 else 1)
            t = _time_graph(run, args.reps, args.iters)
            fl = 2.0 * M * N * K * nw
            by = 2.0 * (N * K * nw + M * K) + out_bytes
            print(f"gemm {name:8s} M={M:6d} N={N:6d} K={K:6d} {t * 1e6:9.1f} us {fl / t / 1e12:8.1f} TFLOP/s "
                  f"{by / t / 1e9:8.1f} GB/s  error_flag={int(flag.item())}")


def bench_attention(args):
    """Back-to-back launches over rotating KV copies (together larger than L2)."""
    d, hq, hkv, dh, ffn, vocab = SHAPES[args.shape]
    rows, vis, nq = args.rows, args.vis, args.nq
    cap = rows * vis
    copies = max(2, -(-(320 << 20) // (cap * hkv * dh * 4)))
    kcs = [torch.randn(cap, hkv, dh, device="cuda").bfloat16() for _ in range(copies)]
    vcs = [torch.randn(cap, hkv, dh, device="cuda").bfloat16() for _ in range(copies)]
    M = rows * nq
    qkv = torch.randn(M, (hq + 2 * hkv) * dh, device="cuda").bfloat16()
    cu_q = torch.arange(0, rows + 1, dtype=torch.int32, device="cuda") * nq
    kv_base = torch.arange(0, rows, dtype=torch.int32, device="cuda") * vis
    visd = torch.full((rows,), vis, dtype=torch.int32, device="cuda")
    scratch = torch.empty(16 << 20, dtype=torch.float32, device="cuda")
    plan = B.attention_plan(cu_q, visd, hq, hkv, dh)
    out = torch.empty(M, hq * dh, dtype=torch.bfloat16, device="cuda")
    def run(i):
        B.op_attention(qkv, kcs[i % copies], vcs[i % copies], cu_q, kv_base, visd, hq, hkv, dh, scratch=scratch,
                       plan=plan, out=out)

    t = _time_graph(run, args.reps, args.iters)
    by = 2.0 * (2.0 * rows * vis * hkv * dh + 2.0 * M * hq * dh)
    fl = 4.0 * rows * nq * vis * hq * dh
    print(f"attention {args.shape} rows={rows} n_q={nq} vis={vis} {t * 1e6:9.1f} us {fl / t / 1e12:8.1f} TFLOP/s "
          f"{by / t / 1e9:8.1f} GB/s")


def bench_confidence(args):
    z = torch.randn(args.rows, args.vocab, device="cuda") * 4
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    t = _time(lambda: B.op_confidence(z, args.vocab - 1), args.iters, flush)
    print(f"confidence rows={args.rows} vocab={args.vocab} {t * 1e6:9.1f} us {4.0 * z.numel() / t / 1e9:8.1f} GB/s")


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("--shape", default="dream", choices=list(SHAPES))
    g.add_argument("--m", type=int, nargs="+", default=[32, 128, 256, 512, 2048, 8192])
    g.add_argument("--only", nargs="*")
    g.add_argument("--hot", action="store_true", help="one weight copy: launches after the first find it in L2")
    g.add_argument("--reps", type=int, default=16, help="back-to-back launches per timing")
    a = sub.add_parser("attention")
    a.add_argument("--shape", default="dream", choices=list(SHAPES))
    a.add_argument("--rows", type=int, default=16)
    a.add_argument("--vis", type=int, default=640)
    a.add_argument("--nq", type=int, default=32)
    a.add_argument("--reps", type=int, default=16)
    c = sub.add_parser("confidence")
    c.add_argument("--rows", type=int, default=512)
    c.add_argument("--vocab", type=int, default=152064)
    for s in (g, a, c):
        s.add_argument("--iters", type=int, default=7)
    args = ap.parse_args()
    torch.manual_seed(0)
    {"gemm": bench_gemm, "attention": bench_attention, "confidence": bench_confidence}[args.cmd](args)


if __name__ == "__main__":
    main()
