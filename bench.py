#!/usr/bin/env python
"""Benchmark of the quantized transformer block (repq_block_forward) on B200.

Metric: quantized block tokens/s.  One step = one pass of the whole hot path (LN+quant, QKV GEMM,
QK^T, Softmax+log2, P.V, proj, LN+quant, fc1/GELU, fc2) over one batch of the DeiT-B-shaped seeded
workload (batch 64 x 197 tokens, dim 768, W4A4).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 (launched by torch.distributed.run) every rank runs its own batch with replicated
parameters: the path shards over the batch with no exchange step (weak scaling, no collective on the
data path).
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
INT8_OVER_BF16 = 2.0          # nominal dense int8 : bf16 tensor throughput on B200
# Fused attention is bound by its per-score arithmetic, not by tensor cores or HBM: pass 1 needs about 8 instructions
# per score (correction, int -> float, scale, max, subtract, scale, ex2, add), pass 2 about 15 (the first three again,
# the code, its power of two, the parity split, packing): the algorithmic count the roofline figure uses.
ATTENTION_INSTR_PER_SCORE = 23

# DRAM traffic of one launch of each stage kernel, from one ncu capture of this file's default workload
# (DeiT-B shape, batch 64; the summaries are under profiles/).  A figure is reported only while the kernel's
# sources still hash to what was captured; otherwise `traffic` is null.
NCU_TRAFFIC_WORKLOAD = ("c2_deit_b", 64)
NCU_TRAFFIC = {   # stage: (DRAM bytes read + written per launch, kernel sources, their sha1 when captured)
    'ln1': (19393280, ['ln_quant.cu', 'f32x2.cuh'], '49b01de9f539'),
    'ln2': (19393280, ['ln_quant.cu', 'f32x2.cuh'], '49b01de9f539'),
    'qkv': (14292480, ['qgemm_tc.cu', 'tc_ptx.cuh', 'epilogue.cuh'], '04dc33d1b726'),
    'attention': (30422016, ['attention_tc.cu', 'tc_ptx.cuh'], 'fbb5e4d22f81'),
    'scores': (85649408, ['scores_tc.cu', 'tc_ptx.cuh'], '0ec10eb039ae'),
    'softmax': (129327104, ['softmax_log2.cu', 'f32x2.cuh'], '9685eb0f7366'),
    'pv': (26712320, ['pv_tc.cu', 'tc_ptx.cuh'], '44d2a2d061d5'),
    'proj': (33026560, ['qgemm_tc.cu', 'tc_ptx.cuh', 'epilogue.cuh'], '04dc33d1b726'),
    'fc1': (20006400, ['qgemm_tc.cu', 'tc_ptx.cuh', 'epilogue.cuh'], '04dc33d1b726'),
    'fc2': (80646912, ['qgemm_tc.cu', 'tc_ptx.cuh', 'epilogue.cuh'], '04dc33d1b726'),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ts, line in self.rows:
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


def measured_traffic(stage, workload, batch):
    """DRAM bytes per launch from the committed ncu capture, or None if it does not describe this run."""
    import hashlib
    if (workload, batch) != NCU_TRAFFIC_WORKLOAD or stage not in NCU_TRAFFIC:
        return None
    nbytes, files, digest = NCU_TRAFFIC[stage]
    h = hashlib.sha1()
    try:
        for f in files:
            h.update(open(os.path.join(ROOT, "paper_2402_05628_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    return nbytes if h.hexdigest()[:12] == digest else None


def stage_costs(cfg, batch):
    """Algorithmic bytes / integer ops of each stage of one block pass (per launch).  Inside the block,
    activation codes and weight codes are stored one per byte (the tensor-core operand format) whatever their
    bit width; only the Softmax codes are packed (two per byte at 4 bits)."""
    B, L, D, H, MLP = batch, cfg["L"], cfg["D"], cfg["H"], cfg["MLP"]
    M, dh = B * L, cfg["D"] // cfg["H"]
    act = 4 if cfg["act"] == "f32" else 2
    ca = 1.0
    cw = 1.0
    cp = 0.5 if cfg["bits_p"] == 4 else 1.0
    n_scores = B * H * L * L * (0.5 if cfg["causal"] else 1.0)

    def gemm(N, K, out_bytes):
        return dict(ops=2.0 * M * N * K, bytes=M * K * ca + N * K * cw + M * N * out_bytes)

    return {
        "ln1": dict(bytes=M * D * (act + ca) + 4 * M, ops=0),
        "qkv": gemm(3 * D, D, ca),
        "scores": dict(ops=2.0 * B * H * L * L * dh, bytes=2 * M * D * ca + n_scores * 4),
        "softmax": dict(bytes=n_scores * (4 + cp), ops=0),
        "pv": dict(ops=2.0 * n_scores * dh, bytes=n_scores * cp + M * D * ca * 2),
        "proj": gemm(D, D, act * 2),          # residual read + output write
        "ln2": dict(bytes=M * D * (act + ca) + 4 * M, ops=0),
        "fc1": gemm(MLP, D, ca),
        "fc2": gemm(D, MLP, act * 2),
    }


def run_reference(args, rank):
    """The CPU oracle, as it stands, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import numpy as np
    from threadpoolctl import threadpool_info
    from oracle import repq_oracle as orc
    from workloads import make_block_inputs
    sample_batch = args.ref_batch
    w = make_block_inputs(args.workload, batch=sample_batch)
    cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    for _ in range(args.warmup):
        orc.block_forward(w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.block_forward(w)
    dt = time.perf_counter() - t0
    tokens = sample_batch * w.cfg["L"] * args.steps
    val = tokens / dt
    from workloads import BLOCK_CONFIGS
    full_batch = BLOCK_CONFIGS[args.workload]["B"]
    sample = "oracle block_forward on %d of the %d batch items per step (float64 numpy)" % (sample_batch, full_batch)
    line = dict(metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * dt / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=args.workload, sample_batch=sample_batch, seq=w.cfg["L"]),
                cpu_baseline=dict(value=val, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_deit_b")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (parity-sized runs)")
    ap.add_argument("--ref-batch", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--staged-attention", action="store_true",
                    help="run scores, Softmax codes and P.V as three kernels instead of the fused attention kernel")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2402_05628_b200.build import build_library
    if local_rank == 0:
        build_library()
    from workloads import make_block_inputs

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    from paper_2402_05628_b200 import binding as B
    from paper_2402_05628_b200.engine import QuantBlock

    from workloads import BLOCK_CONFIGS
    batch = args.batch if args.batch is not None else BLOCK_CONFIGS[args.workload]["B"]
    # replicated parameters, batch sharded over the ranks: generate the global batch, keep this rank's rows
    w = make_block_inputs(args.workload, batch=batch * world)
    cfg = dict(w.cfg)
    cfg["B"] = batch
    L = cfg["L"]
    r0, r1 = shard_rows(world, rank, batch, L)
    w = dataclasses.replace(w, cfg=cfg, x=w.x[r0:r1])
    tokens_per_step = batch * L
    blk = QuantBlock(w, device=dev, staged_attention=args.staged_attention)
    x_host = torch.from_numpy(np.ascontiguousarray(w.x)).to(blk.act_dtype).pin_memory()
    x = x_host.to(dev, non_blocking=True)
    y = torch.empty_like(x, dtype=blk.out_dtype)
    y_host = torch.empty(y.shape, dtype=y.dtype).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > L2 (126 MB)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        blk.forward(x, y)
    barrier()

    # ---- device-resident timing: K steps, L2 flushed between steps, per-step CUDA events on the launch stream
    sampler = ClockSampler(local_rank) if rank == 0 else None
    n0 = B.repq_launch_count()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    t_wall0 = time.time()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)
        starts[i].record(stream)
        blk.forward(x, y)
        ends[i].record(stream)
    barrier()
    t_wall1 = time.time()
    launches = B.repq_launch_count() - n0
    ms_total = sum(s.elapsed_time(e) for s, e in zip(starts, ends))
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None

    # ---- end to end through the host-buffer entry point: every step's input is copied from pinned host memory
    # and its output copied back inside the timed region; the library overlaps the copies of neighbouring steps
    # with the kernels (two device staging buffers per direction)
    y_hosts = [y_host, torch.empty(y.shape, dtype=y.dtype).pin_memory()]
    blk.forward_host([x_host] * 2, y_hosts)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    blk.forward_host([x_host] * args.steps, [y_hosts[i & 1] for i in range(args.steps)])
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    # ---- per-stage timing (CUDA events between stages, same stream) for the roofline figures
    stage_ms = np.zeros(B.REPQ_BLOCK_STAGES)
    n_timed = max(3, min(args.steps, 10))
    for i in range(n_timed):
        flush.fill_(i & 0xFF)
        stage_ms += np.array(blk.forward_timed(x, y))
    stage_ms /= n_timed
    assert B.repq_device_status() == 0, "a bounded device-side wait gave up"

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dev, world)

    if rank == 0:
        peaks = load_peaks()
        costs = stage_costs(cfg, batch)
        stages = {}
        for name, ms in zip(B.BLOCK_STAGE_NAMES, stage_ms):
            c = costs[name]
            st = dict(ms=float(ms), gbs=c["bytes"] / (ms * 1e-3) / 1e9 if ms > 0 else None)
            if c["ops"]:
                st["tops"] = c["ops"] / (ms * 1e-3) / 1e12 if ms > 0 else None
            stages[name] = st
        if not args.staged_attention:
            # the fused kernel ran in the slot of the scores stage; Softmax and P.V have no launch of their own
            att = stages.pop("scores")
            stages.pop("softmax")
            stages.pop("pv")
            n_scores = batch * cfg["H"] * L * L * (0.5 if cfg["causal"] else 1.0)
            att_instr = ATTENTION_INSTR_PER_SCORE * n_scores
            att = dict(ms=att["ms"], gbs=4.0 * batch * L * cfg["D"] / (att["ms"] * 1e-3) / 1e9,
                       ginstr=att_instr / (att["ms"] * 1e-3) / 1e9)
            stages = {k: (att if k == "qkv_next" else v) for k, v in stages.items()}
            ordered = {}
            for k, v in stages.items():
                ordered[k] = v
                if k == "qkv":
                    ordered["attention"] = att
            stages = ordered
        top = max(stages, key=lambda k: stages[k]["ms"])
        int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
        if top in ("qkv", "proj", "fc1", "fc2"):          # scores: bound by its float32 writes, see the HBM branch
            roof = dict(kernel=top, bound="tensor", achieved=stages[top]["tops"], peak=int8_peak, unit="TOP/s",
                        frac=stages[top]["tops"] / int8_peak, traffic=measured_traffic(top, cfg["name"], batch),
                        peak_source="%s bf16 burst x %.0f (nominal int8:bf16)" % (peaks["source"], INT8_OVER_BF16))
        elif top == "attention":
            alu_peak = 148 * 4 * 32 * (clocks["sm_max_mhz"] or 1965.0) * 1e6 / 1e9      # G thread-instructions / s
            roof = dict(kernel=top, bound="alu", achieved=stages[top]["ginstr"], peak=alu_peak, unit="Ginstr/s",
                        frac=stages[top]["ginstr"] / alu_peak, traffic=measured_traffic(top, cfg["name"], batch),
                        peak_source="148 SMs x 4 schedulers x 32 lanes x SM clock; %d instructions per score (two passes)"
                                    % ATTENTION_INSTR_PER_SCORE)
        elif top == "pv":
            roof = dict(kernel=top, bound="tensor", achieved=2 * stages[top]["tops"], peak=peaks["bf16_tflops"],
                        unit="TFLOP/s", frac=2 * stages[top]["tops"] / peaks["bf16_tflops"], traffic=measured_traffic(top, cfg["name"], batch),
                        peak_source="%s bf16 burst; even/odd split doubles the MMA work" % peaks["source"])
        else:
            roof = dict(kernel=top, bound="hbm", achieved=stages[top]["gbs"], peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=stages[top]["gbs"] / peaks["hbm_gbs"], traffic=measured_traffic(top, cfg["name"], batch), peak_source=peaks["source"])
        value = world * tokens_per_step * args.steps / (ms_total * 1e-3)
        e2e_val = world * tokens_per_step * args.steps / (ms_e2e * 1e-3)
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_total / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="u8" if cfg["bits_a"] != 4 else "u4/u8->s32", data="synthetic",
                    config=dict(workload=cfg["name"], batch_per_gpu=batch, seq=L, dim=cfg["D"], heads=cfg["H"],
                                mlp=cfg["MLP"], bits="W%dA%d" % (cfg["bits_w"], cfg["bits_a"]), bits_p=cfg["bits_p"],
                                act=cfg["act"], parallelism="batch-sharded replicas x%d" % world,
                                l2="256 MiB written between timed steps"),
                    clocks=clocks, gpu_launches=int(launches),
                    e2e=dict(value=e2e_val, unit=UNIT, h2d_bytes_per_step=x_host.numel() * x_host.element_size(),
                             d2h_bytes_per_step=y_host.numel() * y_host.element_size()),
                    roofline=roof, stages=stages)
        if world == 1 and not args.no_cpu_baseline:
            from threadpoolctl import threadpool_info
            from oracle import repq_oracle as orc
            nb = max(1, min(batch, 32, 6400 // L))        # bounded sample: roughly 10-30 s of host work
            w_s = make_block_inputs(args.workload, batch=nb)
            orc.block_forward(make_block_inputs(args.workload, batch=1))
            t0 = time.perf_counter()
            reps = 0
            while reps < 1 or time.perf_counter() - t0 < 10.0:
                orc.block_forward(w_s)
                reps += 1
            dt = time.perf_counter() - t0
            cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
            line["cpu_baseline"] = dict(value=nb * L * reps / dt, unit=UNIT, cores=cores, kind="oracle",
                                        sample="%d pass(es) of the float64 numpy oracle block over %d of the %d batch items"
                                               % (reps, nb, batch))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
