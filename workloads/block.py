"""Seeded transformer-block workloads (ViT-S / DeiT-B / ViT-L / LLaMA-7B shaped).

A block workload is: the block input x, the full-precision parameters of the
block, and the clipping bounds that a calibration pass would hand to the
quantizers.  The calibration pass is a stand-in for the paper's calibration
data and per-channel dual clipping: a seeded batch is pushed through a plain
full-precision forward built from PyTorch CPU library calls, and 0.1 / 99.9
percentiles of each activation become its bounds (per channel for the two
LayerNorm activations, per tensor for the others).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np
import torch

from .kernels import affine_params, channel_profile, ln_inputs, percentile_bounds, to_bf16_grid

BLOCK_CONFIGS: Dict[str, dict] = {
    # single ViT-S-style block, fp32 activations
    "c1_vit_s": dict(B=1, L=197, D=384, H=6, MLP=1536, bits_a=4, bits_w=4, bits_p=4, act="f32",
                     sigma_c=1.0, outlier_frac=0.02, outlier_mul=20.0, massive=0, eps=1e-6,
                     causal=False, calib_samples=32, seed=0),
    # DeiT-B-style block, batch 64, bf16 activations (W4A4; the W6A6 variant changes bits only)
    "c2_deit_b": dict(B=64, L=197, D=768, H=12, MLP=3072, bits_a=4, bits_w=4, bits_p=4, act="bf16",
                      sigma_c=1.0, outlier_frac=0.01, outlier_mul=50.0, massive=0, eps=1e-6,
                      causal=False, calib_samples=32, seed=1),
    "c2_deit_b_w6a6": dict(B=64, L=197, D=768, H=12, MLP=3072, bits_a=6, bits_w=6, bits_p=6, act="bf16",
                           sigma_c=1.0, outlier_frac=0.01, outlier_mul=50.0, massive=0, eps=1e-6,
                           causal=False, calib_samples=32, seed=1),
    # ViT-L-style block at 384x384 (577 tokens)
    "c3_vit_l": dict(B=32, L=577, D=1024, H=16, MLP=4096, bits_a=4, bits_w=4, bits_p=4, act="bf16",
                     sigma_c=1.5, outlier_frac=0.005, outlier_mul=100.0, massive=0, eps=1e-6,
                     causal=False, calib_samples=8, seed=2),
    # LLaMA-7B-shaped decoder layer (the paper's block form, causal Softmax, 8-bit log codes)
    "c4_llama7b": dict(B=4, L=2048, D=4096, H=32, MLP=11008, bits_a=4, bits_w=4, bits_p=8, act="bf16",
                       sigma_c=1.0, outlier_frac=0.0, outlier_mul=1.0, massive=4, eps=1e-5,
                       causal=True, calib_samples=1, seed=3),
    # the same shapes in the LLaMA block form: RMSNorm (no shift), rotary embedding on Q and K, gated MLP
    # (w_fc1 = [gate; up] stacked on the output axis, w_fc2 = down), no biases
    "c4_llama7b_arch": dict(B=4, L=2048, D=4096, H=32, MLP=11008, bits_a=4, bits_w=4, bits_p=8, act="bf16",
                            sigma_c=1.0, outlier_frac=0.0, outlier_mul=1.0, massive=4, eps=1e-5,
                            causal=True, calib_samples=1, seed=3, arch="llama", rope_base=10000.0),
}


def block_config(name: str, **overrides) -> dict:
    cfg = dict(BLOCK_CONFIGS[name])
    cfg["name"] = name
    cfg.update(overrides)
    return cfg


@dataclasses.dataclass
class BlockInputs:
    cfg: dict
    x: np.ndarray                # [B*L, D] float32 (on the bf16 grid for bf16 configs)
    ln1_gamma: np.ndarray
    ln1_beta: np.ndarray
    ln1_lo: np.ndarray           # per-channel clipping bounds of LayerNorm-1 activations
    ln1_hi: np.ndarray
    w_qkv: np.ndarray            # [3D, D] rows = output features (q | k | v)
    b_qkv: np.ndarray
    w_proj: np.ndarray           # [D, D]
    b_proj: np.ndarray
    ln2_gamma: np.ndarray
    ln2_beta: np.ndarray
    ln2_lo: np.ndarray
    ln2_hi: np.ndarray
    w_fc1: np.ndarray            # [MLP, D]; LLaMA block form: [2 MLP, D] = gate rows, then up rows
    b_fc1: np.ndarray
    w_fc2: np.ndarray            # [D, MLP]
    b_fc2: np.ndarray
    bounds: Dict[str, tuple]     # 'q','k','v','attn','hidden' -> (lo, hi) float32 scalars
    softmax_scale: float         # scale s of the log-sqrt2 quantizer


def _rotary(t, n, L, H, dh, base):
    """Rotary position embedding through torch's complex multiply: consecutive channel pairs of a head are one
    complex number, rotated by position * base^(-2i/d_h)."""
    theta = torch.pow(torch.tensor(base, dtype=torch.float64), -torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = torch.arange(L, dtype=torch.float64)[:, None] * theta[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)                       # [L, dh/2]
    tc = torch.view_as_complex(t.double().reshape(n, L, H, dh // 2, 2).contiguous())
    return torch.view_as_real(tc * rot[None, :, None, :]).reshape(n, L, H * dh).to(t.dtype)


def _fp_forward(x, p, cfg, want_attn_stats: bool = False):
    """Plain full-precision block forward on CPU (library calls only). x: [n_samples, L, D]."""
    F = torch.nn.functional
    D, H = cfg["D"], cfg["H"]
    dh = D // H
    n, L, _ = x.shape
    llama = cfg.get("arch", "vit") == "llama"

    def norm(t, g, b):
        if llama:
            return F.rms_norm(t, (D,), weight=g, eps=cfg["eps"]) + b
        return F.layer_norm(t, (D,), g, b, cfg["eps"])

    x1 = norm(x, p["ln1_gamma"], p["ln1_beta"])
    qkv = F.linear(x1, p["w_qkv"], p["b_qkv"])
    q, k, v = qkv.split(D, dim=-1)
    if llama:
        q = _rotary(q, n, L, H, dh, cfg.get("rope_base", 10000.0))
        k = _rotary(k, n, L, H, dh, cfg.get("rope_base", 10000.0))
    qh = q.reshape(n, L, H, dh).transpose(1, 2)
    kh = k.reshape(n, L, H, dh).transpose(1, 2)
    vh = v.reshape(n, L, H, dh).transpose(1, 2)
    s = torch.matmul(qh, kh.transpose(-1, -2)) / math.sqrt(dh)
    if cfg["causal"]:
        mask = torch.ones(L, L, dtype=torch.bool).tril()
        s = s.masked_fill(~mask, float("-inf"))
    a = torch.softmax(s, dim=-1)
    if want_attn_stats:
        return a.amax(dim=-1)
    o = torch.matmul(a, vh).transpose(1, 2).reshape(n, L, D)
    xbar = F.linear(o, p["w_proj"], p["b_proj"]) + x
    x2 = norm(xbar, p["ln2_gamma"], p["ln2_beta"])
    h = F.linear(x2, p["w_fc1"], p["b_fc1"])
    if llama:
        gate, up = h.split(cfg["MLP"], dim=-1)
        h = F.silu(gate) * up
    else:
        h = F.gelu(h)
    return dict(x1=x1, q=q, k=k, v=v, attn=o, x2=x2, hidden=h)


def make_block_inputs(name: str, batch: Optional[int] = None, **overrides) -> BlockInputs:
    """Build the seeded workload `name` (optionally with a smaller batch for CPU-sized tests)."""
    cfg = block_config(name, **overrides)
    if batch is not None:
        cfg["B"] = batch
    rng = np.random.default_rng(cfg["seed"])
    B, L, D, MLP = cfg["B"], cfg["L"], cfg["D"], cfg["MLP"]
    bf16 = cfg["act"] == "bf16"

    c, shift = channel_profile(rng, D, cfg["sigma_c"], cfg["outlier_frac"], cfg["outlier_mul"],
                               cfg["massive"])
    g1, b1 = affine_params(rng, D)
    g2, b2 = affine_params(rng, D)
    llama = cfg.get("arch", "vit") == "llama"
    n_fc1 = 2 * MLP if llama else MLP           # gated MLP: gate and up projections stacked

    def weight(n_out, n_in):
        w = rng.standard_normal(size=(n_out, n_in), dtype=np.float32)
        w *= np.float32(0.02)
        return w

    w_qkv = weight(3 * D, D)
    b_qkv = rng.normal(0.0, 0.02, size=3 * D).astype(np.float32)
    w_proj = weight(D, D)
    b_proj = rng.normal(0.0, 0.02, size=D).astype(np.float32)
    w_fc1 = weight(n_fc1, D)
    b_fc1 = rng.normal(0.0, 0.02, size=n_fc1).astype(np.float32)
    w_fc2 = weight(D, MLP)
    b_fc2 = rng.normal(0.0, 0.02, size=D).astype(np.float32)
    if llama:                                    # RMSNorm has no shift, the linear layers no bias
        for a in (b1, b2, b_qkv, b_proj, b_fc1, b_fc2):
            a[...] = 0.0

    # calibration batch first (fixed size), then the benchmark batch: changing B never changes parameters
    n_cal = cfg["calib_samples"]
    x_cal = ln_inputs(rng, n_cal * L, c, shift, bf16).reshape(n_cal, L, D)
    x = ln_inputs(rng, B * L, c, shift, bf16)

    tp = lambda a: torch.from_numpy(a)
    p = dict(ln1_gamma=tp(g1), ln1_beta=tp(b1), w_qkv=tp(w_qkv), b_qkv=tp(b_qkv), w_proj=tp(w_proj),
             b_proj=tp(b_proj), ln2_gamma=tp(g2), ln2_beta=tp(b2), w_fc1=tp(w_fc1), b_fc1=tp(b_fc1),
             w_fc2=tp(w_fc2), b_fc2=tp(b_fc2))

    with torch.no_grad():
        # Attention temperature: scale the query projection so Softmax rows are heavy-tailed
        # (median top-1 probability about 0.5), found by bisection on a slice of the calibration batch.
        xs = tp(x_cal[:1, : min(L, 256)])
        cfg_s = dict(cfg)
        lo_t, hi_t = 0.0, 14.0   # log2 of the temperature
        base_wq = p["w_qkv"][:D].clone()
        base_bq = p["b_qkv"][:D].clone()
        for _ in range(24):
            mid = 0.5 * (lo_t + hi_t)
            p["w_qkv"][:D] = base_wq * (2.0 ** mid)
            p["b_qkv"][:D] = base_bq * (2.0 ** mid)
            top1 = _fp_forward(xs, p, cfg_s, want_attn_stats=True)
            if float(top1.median()) < 0.5:
                lo_t = mid
            else:
                hi_t = mid
        tau = np.float32(2.0 ** (0.5 * (lo_t + hi_t)))
        w_qkv[:D] *= tau
        b_qkv[:D] *= tau
        p["w_qkv"] = tp(w_qkv)
        p["b_qkv"] = tp(b_qkv)

        acts = _fp_forward(tp(x_cal), p, cfg)

    def sub(a, limit=4_000_000):
        a = a.reshape(-1).numpy()
        if a.size > limit:
            a = a[:: a.size // limit + 1]
        return a

    ln1_lo, ln1_hi = percentile_bounds(acts["x1"].reshape(-1, D).numpy(), axis=0)
    ln2_lo, ln2_hi = percentile_bounds(acts["x2"].reshape(-1, D).numpy(), axis=0)
    bounds = {}
    for key in ("q", "k", "v", "attn", "hidden"):
        lo, hi = percentile_bounds(sub(acts[key]))
        bounds[key] = (np.float32(lo), np.float32(hi))

    return BlockInputs(cfg=cfg, x=x, ln1_gamma=g1, ln1_beta=b1, ln1_lo=ln1_lo, ln1_hi=ln1_hi,
                       w_qkv=w_qkv, b_qkv=b_qkv, w_proj=w_proj, b_proj=b_proj,
                       ln2_gamma=g2, ln2_beta=b2, ln2_lo=ln2_lo, ln2_hi=ln2_hi,
                       w_fc1=w_fc1, b_fc1=b_fc1, w_fc2=w_fc2, b_fc2=b_fc2,
                       bounds=bounds, softmax_scale=1.0)
