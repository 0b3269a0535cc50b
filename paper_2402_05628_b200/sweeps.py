"""Kernel-level sweeps (LN+quant, Softmax+log2, integer GEMM, P.V, scores) on one GPU.

Each case times one entry point alone: `reps` back-to-back launches bracketed by CUDA events on the
launch stream, rotating over enough independent input/output buffers that the bytes touched between two
uses of the same buffer exceed the L2 capacity.  Reports achieved GB/s or TOP/s against the algorithmic
bytes / operations of the case.  Inputs are seeded torch tensors with the value ranges of the workloads
(the arithmetic does not depend on the values; parity is checked elsewhere).

    python -m paper_2402_05628_b200.sweeps ln softmax gemm [--quick] [--dim D] [--rows R]
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import binding as B

L2_BYTES = 126 << 20


def _time(fn, n_buf, reps=20, warmup=3):
    st = torch.cuda.current_stream()
    for i in range(warmup):
        fn(i % n_buf)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(st)
    for i in range(reps):
        fn(i % n_buf)
    e1.record(st)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps * 1e-3


def _nbuf(bytes_per_call):
    return max(2, min(64, int(2 * L2_BYTES / max(bytes_per_call, 1)) + 1))


def sweep_ln(quick, only_dim=None, only_rows=None):
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(4)
    out = []
    rows_list = [1024, 16384, 262144] if quick else [1024, 4096, 16384, 65536, 262144, 1048576]
    for D in (384, 768, 1024, 4096, 8192):
        for rows in rows_list:
            if rows * D * 2 > (8 << 30) or (only_dim and D != only_dim) or (only_rows and rows != only_rows):
                continue
            for bits in ((4,) if quick else (4, 6, 8)):
                for dt in (torch.bfloat16,):
                    in_b = rows * D * 2
                    out_b = rows * (D // 2 if bits == 4 else D)
                    n = _nbuf(in_b + out_b)
                    xs = [torch.randn(rows, D, device=dev, generator=g, dtype=torch.float32).to(dt) for _ in range(n)]
                    ld = B.code_row_bytes(D, bits)
                    cs = [torch.empty(rows, ld, dtype=torch.uint8, device=dev) for _ in range(n)]
                    rs = torch.empty(rows, dtype=torch.int32, device=dev)
                    gam = torch.ones(D, device=dev)
                    bet = torch.zeros(D, device=dev)
                    t = _time(lambda i: B.repq_ln_quant(xs[i], gam, bet, 1e-6, 0.25, 7, bits, cs[i], rs), n)
                    byt = in_b + out_b + 4 * rows
                    out.append(dict(kernel="ln_quant", rows=rows, D=D, bits=bits, dtype="bf16", us=t * 1e6,
                                    gbs=byt / t / 1e9, tokens_per_s=rows / t))
                    del xs, cs
    return out


def sweep_softmax(quick, only_dim=None, only_rows=None):
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(4)
    out = []
    for L in (197, 577, 2048, 8192):
        if only_dim and L != only_dim:
            continue
        for rows in ((151296,) if quick else (4096, 32768, 151296)):
            if L >= 2048:
                rows = min(rows, 32768)
            for bits in (4, 8):
                ld = (L + 3) // 4 * 4
                unit = 4 if bits == 4 else 8
                ldc = max(B.code_row_bytes(L, bits), (L + 7) // 8 * unit)
                byt = rows * L * 4 + rows * (L // 2 if bits == 4 else L)
                n = _nbuf(byt)
                ss = [torch.randn(rows, ld, device=dev, generator=g) * 4 for _ in range(n)]
                cs = [torch.empty(rows, ldc, dtype=torch.uint8, device=dev) for _ in range(n)]
                t = _time(lambda i: B.repq_softmax_log2(ss[i], L, 1.0, bits, cs[i]), n)
                out.append(dict(kernel="softmax_log2", rows=rows, L=L, bits=bits, dtype="f32", us=t * 1e6,
                                gbs=byt / t / 1e9))
                del ss, cs
    return out


def sweep_gemm(quick, only_dim=None, only_rows=None):
    dev = torch.device("cuda:0")
    out = []
    shapes = [(12608, 2304, 768), (12608, 768, 768), (12608, 3072, 768), (12608, 768, 3072),
              (16384, 4096, 4096), (8192, 12288, 4096), (8192, 11008, 4096), (8192, 4096, 11008)]
    if not quick:
        shapes += [(2048, 768, 768), (2048, 4096, 4096), (65536, 768, 768), (65536, 4096, 4096), (18464, 4096, 1024)]
    for (M, N, K) in shapes:
        for bits in (4, 8):
            for kind in ("bf16", "codes"):
                lda = B.code_row_bytes(K, bits)
                a = torch.randint(0, 256, (M, lda), dtype=torch.uint8, device=dev)
                w = torch.randint(0, 256, (N, lda), dtype=torch.uint8, device=dev)
                if bits == 6:
                    a &= 63
                    w &= 63
                s_w = torch.full((N,), 0.01, device=dev)
                z_w = torch.full((N,), 7, dtype=torch.int32, device=dev)
                bias = torch.zeros(N, device=dev)
                asum = torch.zeros(M, dtype=torch.int32, device=dev)
                wsum = torch.zeros(N, dtype=torch.int32, device=dev)
                if kind == "bf16":
                    o = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
                    d = B.gemm_desc(M, N, K, a, bits, 0.1, 7, w, bits, o, s_w=s_w, z_w=z_w, bias=bias, a_row_sum=asum,
                                    w_row_sum=wsum, out_kind=B.REPQ_OUT_BF16)
                else:
                    o = torch.empty(M, B.code_row_bytes(N, bits), dtype=torch.uint8, device=dev)
                    d = B.gemm_desc(M, N, K, a, bits, 0.1, 7, w, bits, o, s_w=s_w, z_w=z_w, bias=bias, a_row_sum=asum,
                                    w_row_sum=wsum, out_kind=B.REPQ_OUT_CODES, out_bits=bits, out_scale=[0.5],
                                    out_zero=[7])
                ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)
                t = _time(lambda i: B.repq_qgemm(d, ws), 1, reps=10)
                out.append(dict(kernel="qgemm", M=M, N=N, K=K, bits="W%dA%d" % (bits, bits), out=kind, us=t * 1e6,
                                tops=2.0 * M * N * K / t / 1e12))
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("which", nargs="+", choices=["ln", "softmax", "gemm"])
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--dim", type=int, default=None, help="only this feature size (ln) / row length (softmax)")
    ap.add_argument("--rows", type=int, default=None, help="only this row count (ln)")
    args = ap.parse_args()
    B.lib()
    for name in args.which:
        for row in {"ln": sweep_ln, "softmax": sweep_softmax, "gemm": sweep_gemm}[name](args.quick, args.dim, args.rows):
            print(json.dumps(row))
            sys.stdout.flush()


if __name__ == "__main__":
    main()
