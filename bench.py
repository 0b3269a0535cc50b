#!/usr/bin/env python
"""Benchmark of the quantized transformer block (repq_block_forward) on B200.

Metric: quantized block tokens/s.  One step = one pass of the whole hot path (LN+quant, QKV GEMM, fused attention
= QK^T + Softmax/log2 codes + P.V, proj, LN+quant, fc1/GELU, fc2) over one batch of a seeded synthetic workload.
The headline workload is the largest single-GPU configuration, the LLaMA-7B-shaped layer (batch 4 x 2048 tokens,
dim 4096, 32 heads, MLP 11008, causal, W4A4 with 8-bit log codes).  Prints ONE JSON line, which also carries

  workloads   the same measurement (tokens/s, ms per pass, end-to-end, per-stage roofline fractions) on the other
              block configurations: ViT-S, DeiT-B (W4A4 and W6A6), ViT-L/384, and the LLaMA block form
  kernels     single-kernel sweep points: fused LN+quant and Softmax+log2 as a fraction of the HBM copy rate, the
              integer GEMM as a fraction of the int8 tensor-core peak
  sustained   the headline block looped for seconds, with the SM clock seen while it ran

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 every rank (one per GPU; spawned here through torch.distributed.run unless the launcher already did)
runs its own batch with replicated parameters: the path shards over the batch with no exchange step (weak
scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "quantized_block_tokens_per_s"
UNIT = "tokens/s"
HEADLINE = "c4_llama7b"
OTHER_WORKLOADS = ("c1_vit_s", "c2_deit_b", "c2_deit_b_w6a6", "c3_vit_l", "c4_llama7b_arch")
INT8_OVER_BF16 = 2.0          # nominal dense int8 : bf16 tensor throughput on B200
L2_BYTES = 126 << 20
# Own model of the fused attention kernel's arithmetic, kept as a side figure from the first version of the kernel: about
# 8 thread instructions per score in the statistics pass (int -> float, scale, max, subtract, ex2, add) and 15 in the code
# pass.  (The present kernel needs about half of that and is not bound by it.)
ATTENTION_INSTR_PER_SCORE = 23

# DRAM traffic of one launch of a stage kernel, from one ncu capture of the same bench command (summaries under
# profiles/).  A figure is reported only while the kernel's sources still hash to what was captured.
NCU_TRAFFIC = {   # (workload, batch, stage): (DRAM bytes read + written per launch, kernel sources, their sha1 when captured)
    ("c4_llama7b", 4, "attention"): (138199296, ["attention_tc.cu", "tc_ptx.cuh"], "47dd87935b26"),
    ("c4_llama7b", 4, "qkv"): (166124032, ["qgemm_tc.cu", "tc_ptx.cuh", "epilogue.cuh"], "f76285585384"),
    ("c4_llama7b", 4, "proj"): (201283840, ["qgemm_tc.cu", "tc_ptx.cuh", "epilogue.cuh"], "f76285585384"),
    ("c4_llama7b", 4, "fc1"): (148836608, ["qgemm_tc.cu", "tc_ptx.cuh", "epilogue.cuh"], "f76285585384"),
    ("c4_llama7b", 4, "fc2"): (517648896, ["qgemm_tc.cu", "tc_ptx.cuh", "epilogue.cuh"], "f76285585384"),
    ("c4_llama7b", 4, "ln1"): (71826432, ["ln_quant.cu", "f32x2.cuh"], "1eacf83c9513"),
    ("c4_llama7b", 4, "ln2"): (71635712, ["ln_quant.cu", "f32x2.cuh"], "1eacf83c9513"),
    ("c2_deit_b", 64, "attention"): (29160192, ["attention_tc.cu", "tc_ptx.cuh"], "47dd87935b26"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 25):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", str(period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def window(self, t0: float, t1: float):
        """Median SM clock and the throttle reasons seen between t0 and t1 (wall clock)."""
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"], samples=0)
        sm, mx, reasons = [], None, set()
        for ts, line in list(self.rows):
            if ts < t0 - 0.05 or ts > t1 + 0.15:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        med = sm[len(sm) // 2] if sm else None
        return dict(sm_mhz=med, sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))

    def stop(self):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()


def shard_rows(world: int, rank: int, batch_per_gpu: int, seq: int):
    """Rows of the global batch (world * batch_per_gpu items) that rank `rank` owns: the path shards over the
    batch with no exchange step, so a rank's shard is a contiguous block of whole batch items."""
    rows = batch_per_gpu * seq
    return rank * rows, (rank + 1) * rows


def max_over_ranks(values, device, world: int):
    """Element-wise MAX of a list of floats over all ranks (timings are reported as the slowest rank's)."""
    if world == 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def spawn_command(n_gpus: int, argv, port: int):
    """The launch of N ranks on this node (one process per GPU) when the caller did not provide them."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def measured_traffic(stage, workload, batch):
    """DRAM bytes per launch from the committed ncu capture, or None if it does not describe this run."""
    import hashlib
    key = (workload, batch, stage)
    if key not in NCU_TRAFFIC:
        return None
    nbytes, files, digest = NCU_TRAFFIC[key]
    h = hashlib.sha1()
    try:
        for f in files:
            h.update(open(os.path.join(ROOT, "paper_2402_05628_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    return nbytes if h.hexdigest()[:12] == digest else None


def stage_costs(cfg, batch):
    """Algorithmic bytes / operations of each stage of one block pass (per launch).  Inside the block, activation
    codes and weight codes are stored one per byte (the tensor-core operand format) whatever their bit width; only
    the Softmax codes of the separate attention stages are packed (two per byte at 4 bits)."""
    B, L, D, H, MLP = batch, cfg["L"], cfg["D"], cfg["H"], cfg["MLP"]
    M, dh = B * L, cfg["D"] // cfg["H"]
    act = 4 if cfg["act"] == "f32" else 2
    ca = cw = 1.0
    cp = 0.5 if cfg["bits_p"] == 4 else 1.0
    n_scores = B * H * L * L * (0.5 if cfg["causal"] else 1.0)
    llama = cfg.get("arch", "vit") == "llama"

    def gemm(N, K, out_bytes, n_out=None):
        return dict(ops=2.0 * M * N * K, bytes=M * K * ca + N * K * cw + M * (n_out or N) * out_bytes)

    return {
        "ln1": dict(bytes=M * D * (act + ca) + 4 * M, ops=0),
        "qkv": gemm(3 * D, D, ca),
        "scores": dict(ops=2.0 * n_scores * dh, bytes=2 * M * D * ca + n_scores * 4),
        "softmax": dict(bytes=n_scores * (4 + cp), ops=0),
        "pv": dict(ops=2.0 * n_scores * dh, bytes=n_scores * cp + M * D * ca * 2),
        # fused attention: Q, K, V codes in, attention codes out; one int8 and one bf16 contraction
        "attention": dict(bytes=4 * M * D * ca, ops_i8=2.0 * n_scores * dh, flop_bf16=2.0 * n_scores * dh, scores=n_scores),
        "proj": gemm(D, D, act * 2),          # residual read + output write
        "ln2": dict(bytes=M * D * (act + ca) + 4 * M, ops=0),
        "fc1": gemm(2 * MLP, D, ca, MLP) if llama else gemm(MLP, D, ca),
        "fc2": gemm(D, MLP, act * 2),
    }


def stage_record(name, ms, cost, peaks, sm_max_mhz):
    """Achieved rates of one stage and its fractions of the rooflines that could bound it."""
    if not ms or ms <= 0:
        return dict(ms=ms)
    t = ms * 1e-3
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    rec = dict(ms=float(ms), gbs=cost["bytes"] / t / 1e9, frac_hbm=cost["bytes"] / t / 1e9 / peaks["hbm_gbs"])
    if name == "attention":
        tensor_s = cost["ops_i8"] / (int8_peak * 1e12) + cost["flop_bf16"] / (peaks["bf16_tflops"] * 1e12)
        alu_peak = 148 * 4 * 32 * (sm_max_mhz or 1965.0) * 1e6
        rec.update(bf16_equiv_tflops=(cost["ops_i8"] / INT8_OVER_BF16 + cost["flop_bf16"]) / t / 1e12,
                   frac_tensor=tensor_s / t,
                   frac_issue_model=ATTENTION_INSTR_PER_SCORE * cost["scores"] / t / alu_peak)
    elif cost.get("ops"):
        rec["tops"] = cost["ops"] / t / 1e12
        if name in ("qkv", "proj", "fc1", "fc2"):
            rec["frac_int8_peak"] = rec["tops"] / int8_peak
        elif name == "pv":
            rec["frac_bf16_peak"] = rec["tops"] / peaks["bf16_tflops"]
    return rec


def measure_block(name, batch, args, dev, rank, world, peaks, headline, sampler=None):
    """Device-resident timing (K steps, L2 flushed between steps), end-to-end timing through the host-buffer entry
    point, and per-stage timing of one block workload on this rank's shard."""
    import numpy as np
    import torch
    from paper_2402_05628_b200 import binding as B
    from paper_2402_05628_b200.engine import QuantBlock
    from workloads import make_block_inputs

    # replicated parameters, batch sharded over the ranks: generate the global batch, keep this rank's rows
    w = make_block_inputs(name, batch=batch * world)
    cfg = dict(w.cfg)
    cfg["B"] = batch
    L = cfg["L"]
    r0, r1 = shard_rows(world, rank, batch, L)
    w = dataclasses.replace(w, cfg=cfg, x=w.x[r0:r1])
    tokens_per_step = batch * L
    blk = QuantBlock(w, device=dev, staged_attention=args.staged_attention, weight_storage=args.weights)
    x_host = torch.from_numpy(np.ascontiguousarray(w.x)).to(blk.act_dtype).pin_memory()
    x = x_host.to(dev, non_blocking=True)
    y = torch.empty_like(x, dtype=blk.out_dtype)
    y_hosts = [torch.empty(y.shape, dtype=y.dtype).pin_memory() for _ in range(2)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > L2 (126 MB)
    stream = torch.cuda.current_stream()
    steps = args.steps

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        blk.forward(x, y)
    barrier()

    # ---- device-resident timing: per-step CUDA events on the launch stream
    n0 = B.repq_launch_count()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier()
    t_wall0 = time.time()
    for i in range(steps):
        flush.fill_(i & 0xFF)
        starts[i].record(stream)
        blk.forward(x, y)
        ends[i].record(stream)
    barrier()
    t_wall1 = time.time()
    launches = B.repq_launch_count() - n0
    ms_total = sum(s.elapsed_time(e) for s, e in zip(starts, ends))
    clocks = sampler.window(t_wall0, t_wall1) if sampler else None

    # ---- end to end through the host-buffer entry point: every step's input is copied from pinned host memory
    # and its output copied back inside the timed region; the library overlaps the copies of neighbouring steps
    # with the kernels (two device staging buffers per direction)
    blk.forward_host([x_host] * 2, y_hosts)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    blk.forward_host([x_host] * steps, [y_hosts[i & 1] for i in range(steps)])
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    # ---- per-stage timing (CUDA events between the stages, same stream; the kernels then run one after the other
    # without the overlap of the free-running block, so the stage times add up to a little more than a pass)
    stage_ms = np.zeros(B.REPQ_BLOCK_STAGES)
    n_timed = max(3, min(steps, 10))
    for i in range(n_timed):
        flush.fill_(i & 0xFF)
        stage_ms += np.array(blk.forward_timed(x, y))
    stage_ms /= n_timed
    assert B.repq_device_status() == 0, "a bounded device-side wait gave up"

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dev, world)
    costs = stage_costs(cfg, batch)
    sm_max = clocks["sm_max_mhz"] if clocks else None
    raw = dict(zip(B.BLOCK_STAGE_NAMES, stage_ms))
    stages = {}
    for st in B.BLOCK_STAGE_NAMES:
        if not args.staged_attention and st in ("softmax", "pv"):
            continue
        key = "attention" if (st == "scores" and not args.staged_attention) else st
        stages[key] = stage_record(key, float(raw[st]), costs[key], peaks, sm_max)
    rec = dict(workload=name, batch_per_gpu=batch, tokens_per_step=tokens_per_step,
               value=world * tokens_per_step * steps / (ms_total * 1e-3), ms_per_step=ms_total / steps,
               e2e=dict(value=world * tokens_per_step * steps / (ms_e2e * 1e-3), unit=UNIT,
                        h2d_bytes_per_step=x_host.numel() * x_host.element_size(),
                        d2h_bytes_per_step=y_hosts[0].numel() * y_hosts[0].element_size()),
               stages=stages, gpu_launches=int(launches), clocks=clocks, cfg=cfg,
               weight_bytes=int(sum(l.codes.numel() for l in (blk.qkv, blk.proj, blk.fc1, blk.fc2))))
    if headline:
        rec["_blk"], rec["_x"], rec["_y"] = blk, x, y
    return rec


def sustained_run(rec, seconds, sampler, dev):
    """The headline block back to back for `seconds`: a steady-state figure under the clocks a long run settles at."""
    import torch
    blk, x, y = rec["_blk"], rec["_x"], rec["_y"]
    stream = torch.cuda.current_stream()
    chunk = max(10, int(0.1 / (rec["ms_per_step"] * 1e-3)))
    torch.cuda.synchronize()
    t0 = time.time()
    n, ms = 0, 0.0
    while time.time() - t0 < seconds:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(chunk):
            blk.forward(x, y)
        e1.record(stream)
        torch.cuda.synchronize()
        ms += e0.elapsed_time(e1)
        n += chunk
    t1 = time.time()
    clocks = sampler.window(t0 + 0.5, t1) if sampler else None
    out = dict(seconds=t1 - t0, steps=n, ms_per_step=ms / n, value=rec["tokens_per_step"] * n / (ms * 1e-3), unit=UNIT,
               clocks=clocks, l2="not flushed (back-to-back passes; the working set exceeds L2)")
    if clocks and clocks.get("sm_mhz"):
        out["ms_times_mhz"] = ms / n * clocks["sm_mhz"]
    return out


# ------------------------------------------------------------------------------------------ single-kernel sweeps

def _time_launches(fn, n_buf, reps=20, warmup=3):
    import torch
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
    """Independent buffer sets to rotate over, so that the bytes touched between two uses of one set exceed L2."""
    return max(2, min(64, int(2 * L2_BYTES / max(bytes_per_call, 1)) + 1))


def kernel_sweeps(peaks, dev, quick=True, only=None, dim=None):
    """Single-kernel points of the sweeps: every case times one entry point alone, `reps` launches bracketed by CUDA
    events, rotating over buffer sets larger than L2.  Inputs are seeded torch tensors with the value ranges of the
    workloads (the kernels' time does not depend on the values; parity is checked in the tests)."""
    import torch
    from paper_2402_05628_b200 import binding as B
    g = torch.Generator(device=dev).manual_seed(4)
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    out = dict(ln_quant=[], softmax_log2=[], qgemm=[], dual_clip=[])
    # per-channel dual clipping (calibration-time; Table X of the paper reports 17 s (DeiT-S) and 46 s (LLaMA-13B) per layer
    # for its PyTorch implementation on an A6000: context, not a target): 100 Adam steps on the activations of a
    # calibration batch, float64, every step one pass over the L2-resident activations
    for n, D in ((6304, 384), (16384, 4096)):
        if only and only != "clip":
            continue
        x = torch.randn(n, D, device=dev, generator=g, dtype=torch.float32) * 2.0 + 0.3
        lo, hi = torch.empty(D, device=dev), torch.empty(D, device=dev)
        t = _time_launches(lambda i: B.repq_dual_clip(x, 4, lo, hi, None, iters=100, lr=0.01, alpha0=2.0), 1, reps=3, warmup=1)
        out["dual_clip"].append(dict(tokens=n, D=D, iters=100, ms=t * 1e3, passes_gbs=102 * n * D * 4 / t / 1e9))
    # fused LN + quant: bf16 in, packed 4-bit codes out (2.5 D bytes per token + 4 for the row sum)
    for D in (384, 768, 1024, 4096, 8192):
        if (only and only != "ln") or (dim and dim != D):
            continue
        rows = 262144
        for bits, label in ((4, "packed 4-bit"), (4 | B.REPQ_BYTE_CODES, "4-bit in bytes")):
            if quick and bits != 4 and D not in (768, 4096):
                continue
            ld = B.code_row_bytes(D, bits)
            byt = rows * D * 2 + rows * (D // 2 if bits == 4 else D) + 4 * rows
            n = _nbuf(byt)
            xs = [torch.randn(rows, D, device=dev, generator=g, dtype=torch.float32).to(torch.bfloat16) for _ in range(n)]
            cs = [torch.empty(rows, ld, dtype=torch.uint8, device=dev) for _ in range(n)]
            rs = torch.empty(rows, dtype=torch.int32, device=dev)
            gam, bet = torch.ones(D, device=dev), torch.zeros(D, device=dev)
            t = _time_launches(lambda i: B.repq_ln_quant(xs[i], gam, bet, 1e-6, 0.25, 7, bits, cs[i], rs), n)
            out["ln_quant"].append(dict(rows=rows, D=D, codes=label, us=t * 1e6, gbs=byt / t / 1e9,
                                        frac_hbm=byt / t / 1e9 / peaks["hbm_gbs"], tokens_per_s=rows / t))
            del xs, cs
    # Softmax + log2 codes: float32 scores in, packed 4-bit / 8-bit codes out
    for L, rows in ((197, 151296), (577, 151296), (2048, 32768), (8192, 32768)):
        if (only and only != "softmax") or (dim and dim != L):
            continue
        for bits in (4, 8):
            ld = (L + 3) // 4 * 4
            ldc = max(B.code_row_bytes(L, bits), (L + 7) // 8 * (4 if bits == 4 else 8))
            byt = rows * L * 4 + rows * (L // 2 if bits == 4 else L)
            n = _nbuf(byt)
            ss = [torch.randn(rows, ld, device=dev, generator=g) * 4 for _ in range(n)]
            cs = [torch.empty(rows, ldc, dtype=torch.uint8, device=dev) for _ in range(n)]
            t = _time_launches(lambda i: B.repq_softmax_log2(ss[i], L, 1.0, bits, cs[i]), n)
            out["softmax_log2"].append(dict(rows=rows, L=L, bits=bits, us=t * 1e6, gbs=byt / t / 1e9,
                                            frac_hbm=byt / t / 1e9 / peaks["hbm_gbs"]))
            del ss, cs
    # integer GEMM at M = 16384 on the layer shapes of the block configurations; operands one code per byte
    # (W4A4: 4-bit quantizers in byte containers, the block's format; W8A8: 8-bit codes), bf16 and code outputs
    M = 16384
    for (N, K) in ((2304, 768), (768, 768), (3072, 768), (768, 3072), (3072, 1024), (4096, 4096), (12288, 4096),
                   (11008, 4096), (4096, 11008)):
        if (only and only != "gemm") or (dim and dim != N):
            continue
        for qbits in (4, 8):
            bits = qbits | B.REPQ_BYTE_CODES
            for kind in ("bf16", "codes"):
                if quick and kind == "bf16" and qbits == 8:
                    continue
                a = torch.randint(0, 1 << qbits, (M, K), dtype=torch.uint8, device=dev, generator=g)
                wq = torch.randint(0, 1 << qbits, (N, K), dtype=torch.uint8, device=dev, generator=g)
                s_w = torch.full((N,), 0.01, device=dev)
                z_w = torch.full((N,), 7, dtype=torch.int32, device=dev)
                bias = torch.zeros(N, device=dev)
                asum = a.sum(dim=1, dtype=torch.int32)
                wsum = wq.sum(dim=1, dtype=torch.int32)
                if kind == "bf16":
                    o = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
                    d = B.gemm_desc(M, N, K, a, bits, 0.1, 7, wq, bits, o, s_w=s_w, z_w=z_w, bias=bias, a_row_sum=asum,
                                    w_row_sum=wsum, out_kind=B.REPQ_OUT_BF16)
                else:
                    o = torch.empty(M, N, dtype=torch.uint8, device=dev)
                    d = B.gemm_desc(M, N, K, a, bits, 0.1, 7, wq, bits, o, s_w=s_w, z_w=z_w, bias=bias, a_row_sum=asum,
                                    w_row_sum=wsum, out_kind=B.REPQ_OUT_CODES, out_bits=bits, out_scale=[0.5], out_zero=[7])
                ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)
                t = _time_launches(lambda i: B.repq_qgemm(d, ws), 1, reps=10)
                tops = 2.0 * M * N * K / t / 1e12
                out["qgemm"].append(dict(M=M, N=N, K=K, bits="W%dA%d" % (qbits, qbits), out=kind, us=t * 1e6, tops=tops,
                                         frac_int8_peak=tops / int8_peak))
    return out


# ------------------------------------------------------------------------------------------ the oracle's arm

def oracle_sample(name, ref_batch, ref_tokens):
    """A bounded sample of workload `name` for the CPU oracle: some of its batch items and, under a causal mask, a
    prefix of the sequence (the outputs of the first tokens do not depend on later ones, so the prefix is what the
    full workload computes for those tokens)."""
    from workloads import BLOCK_CONFIGS, make_block_inputs
    full = BLOCK_CONFIGS[name]
    nb = max(1, min(full["B"], ref_batch))
    w = make_block_inputs(name, batch=nb)
    what = "%d of the %d batch items" % (nb, full["B"])
    if full["causal"] and ref_tokens and ref_tokens < full["L"]:
        cfg = dict(w.cfg)
        cfg["L"] = ref_tokens
        rows = [i * full["L"] + j for i in range(nb) for j in range(ref_tokens)]
        w = dataclasses.replace(w, cfg=cfg, x=w.x[rows])
        what += ", first %d of %d tokens (causal prefix)" % (ref_tokens, full["L"])
    return w, nb * w.cfg["L"], what


def run_reference(args, rank):
    """The CPU oracle, as it stands, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from threadpoolctl import threadpool_info
    from oracle import repq_oracle as orc
    w, tokens, what = oracle_sample(args.workload, args.ref_batch, args.ref_tokens)
    cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    for _ in range(args.warmup):
        orc.block_forward(w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.block_forward(w)
    dt = time.perf_counter() - t0
    val = tokens * args.steps / dt
    sample = "oracle block_forward (float64 numpy) per step on " + what
    line = dict(metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * dt / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=args.workload, sample=what, seq=w.cfg["L"]),
                cpu_baseline=dict(value=val, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (parity-sized runs)")
    ap.add_argument("--ref-batch", type=int, default=1, help="batch items of the oracle's sample")
    ap.add_argument("--ref-tokens", type=int, default=512, help="causal workloads: sequence prefix of the oracle's sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="headline workload only: no other workloads, sweeps or sustained run")
    ap.add_argument("--sustained-seconds", type=float, default=3.0)
    ap.add_argument("--sweep-only", default=None, choices=["ln", "softmax", "gemm", "clip"],
                    help="run only the single-kernel sweep points of this kernel and print them (profiling aid)")
    ap.add_argument("--sweep-dim", type=int, default=None, help="with --sweep-only: only this D (ln), L (softmax) or N (gemm)")
    ap.add_argument("--weights", default="bytes", choices=["packed", "bytes"],
                    help="weight codes in device memory: packed (4-bit two per byte, 6-bit four to three bytes; expanded in shared memory "
                         "by the GEMM) or one per byte")
    ap.add_argument("--staged-attention", action="store_true",
                    help="run scores, Softmax codes and P.V as three kernels instead of the fused attention kernel")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not launched as ranks: start one process per GPU on this node and hand over
        port = 29500 + os.getpid() % 2000
        sys.exit(subprocess.call(spawn_command(args.gpus, sys.argv[1:], port)))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2402_05628_b200.build import build_library
    if local_rank == 0:
        build_library()
    from workloads import BLOCK_CONFIGS

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    from paper_2402_05628_b200 import binding as B
    B.lib()

    peaks = load_peaks()
    if args.sweep_only:
        print(json.dumps(kernel_sweeps(peaks, dev, only=args.sweep_only, dim=args.sweep_dim)))
        return
    sampler = ClockSampler(local_rank) if rank == 0 else None
    batch = args.batch if args.batch is not None else BLOCK_CONFIGS[args.workload]["B"]
    head = measure_block(args.workload, batch, args, dev, rank, world, peaks, headline=True, sampler=sampler)
    extras = world == 1 and not args.no_extras
    sustained = sustained_run(head, args.sustained_seconds, sampler, dev) if extras and args.sustained_seconds > 0 else None
    for k in ("_blk", "_x", "_y"):
        head.pop(k, None)
    torch.cuda.empty_cache()

    others, sweeps = {}, None
    if extras:
        for name in OTHER_WORKLOADS:
            if name == args.workload:
                continue
            r = measure_block(name, BLOCK_CONFIGS[name]["B"], args, dev, rank, world, peaks, headline=False, sampler=sampler)
            c = r.pop("cfg")
            r.pop("clocks", None)
            r["bits"] = "W%dA%d" % (c["bits_w"], c["bits_a"])
            r["unit"] = UNIT
            others[name] = r
            torch.cuda.empty_cache()
        sweeps = kernel_sweeps(peaks, dev)
        torch.cuda.empty_cache()
    if sampler:
        sampler.stop()

    if rank == 0:
        cfg, stages = head["cfg"], head["stages"]
        top = max(stages, key=lambda k: stages[k]["ms"])
        st = stages[top]
        int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
        traffic = measured_traffic(top, cfg["name"], batch)
        if top == "attention":
            # two contractions (int8 QK^T, bf16 P.V): expressed in bf16-equivalent FLOP (an int8 operation counts
            # 1 / INT8_OVER_BF16), so that achieved / peak = (tensor time at the peaks) / (measured time)
            roof = dict(kernel=top, bound="tensor", achieved=st["bf16_equiv_tflops"], peak=peaks["bf16_tflops"], unit="TFLOP/s",
                        frac=st["frac_tensor"], traffic=traffic, frac_hbm=st["frac_hbm"], frac_issue_model=st["frac_issue_model"],
                        peak_source="%s bf16 burst; int8 operations of QK^T counted at 1/%.0f (nominal int8:bf16); algorithmic "
                                    "operation counts (one pass over the keys, P.V once)" % (peaks["source"], INT8_OVER_BF16))
        elif top in ("qkv", "proj", "fc1", "fc2"):
            roof = dict(kernel=top, bound="tensor", achieved=st["tops"], peak=int8_peak, unit="TOP/s", frac=st["frac_int8_peak"],
                        traffic=traffic, frac_hbm=st["frac_hbm"],
                        peak_source="%s bf16 burst x %.0f (nominal int8:bf16)" % (peaks["source"], INT8_OVER_BF16))
        elif top == "pv":
            roof = dict(kernel=top, bound="tensor", achieved=st["tops"], peak=peaks["bf16_tflops"], unit="TFLOP/s",
                        frac=st["frac_bf16_peak"], traffic=traffic, frac_hbm=st["frac_hbm"], peak_source="%s bf16 burst" % peaks["source"])
        else:
            roof = dict(kernel=top, bound="hbm", achieved=st["gbs"], peak=peaks["hbm_gbs"], unit="GB/s", frac=st["frac_hbm"],
                        traffic=traffic, peak_source=peaks["source"])
        line = dict(metric=METRIC, value=head["value"], unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=head["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="u8" if cfg["bits_a"] != 4 else "u4/u8->s32", data="synthetic",
                    config=dict(workload=cfg["name"], batch_per_gpu=batch, seq=cfg["L"], dim=cfg["D"], heads=cfg["H"],
                                mlp=cfg["MLP"], bits="W%dA%d" % (cfg["bits_w"], cfg["bits_a"]), bits_p=cfg["bits_p"],
                                act=cfg["act"], causal=bool(cfg["causal"]), weights=args.weights,
                                weight_code_bytes=head["weight_bytes"], parallelism="batch-sharded replicas x%d" % world,
                                l2="256 MiB written between timed steps",
                                stage_times="CUDA events between the stages: kernels serialised, so their sum exceeds ms_per_step"),
                    clocks=head["clocks"], gpu_launches=head["gpu_launches"], e2e=head["e2e"], roofline=roof, stages=stages,
                    peaks=dict(hbm_gbs=peaks["hbm_gbs"], bf16_tflops=peaks["bf16_tflops"], int8_tops=int8_peak, source=peaks["source"]))
        if sustained:
            line["sustained"] = sustained
        if others:
            line["workloads"] = others
        if sweeps:
            line["kernels"] = sweeps
        if world == 1 and not args.no_cpu_baseline:
            from threadpoolctl import threadpool_info
            from oracle import repq_oracle as orc
            full = BLOCK_CONFIGS[args.workload]
            nb = max(1, min(batch, 32, 3200 // full["L"]))        # bounded sample: roughly 10-30 s of host work
            w_s, tokens, what = oracle_sample(args.workload, nb, None)
            t0 = time.perf_counter()
            reps = 0
            while reps < 1 or time.perf_counter() - t0 < 10.0:
                orc.block_forward(w_s)
                reps += 1
            dt = time.perf_counter() - t0
            cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
            line["cpu_baseline"] = dict(value=tokens * reps / dt, unit=UNIT, cores=cores, kind="oracle",
                                        sample="%d pass(es) of the float64 numpy oracle block over %s" % (reps, what))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
