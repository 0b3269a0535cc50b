"""Kernel-level seeded generators (LayerNorm rows, attention logits, code matrices).

Distribution recipes (stand-ins for activations of trained models, which are
not available offline):

* LayerNorm inputs follow the inter-channel variation the paper shows for
  DeiT-S / LLaMA-7B (Fig. 4): every channel has its own magnitude drawn from a
  log-normal, a small fraction of channels are outliers multiplied by a large
  factor, and every channel carries a mean shift so that per-channel clipping
  bounds are asymmetric (Fig. 8).
* Attention logits give power-law Softmax rows (Fig. 5): one dominant
  probability and a k^-alpha tail.
"""
from __future__ import annotations

import numpy as np
import torch


def to_bf16_grid(a: np.ndarray) -> np.ndarray:
    """Round a float array to the nearest bf16 value, returned as float32 (pure dtype cast)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def channel_profile(rng: np.random.Generator, D: int, sigma_c: float, outlier_frac: float,
                    outlier_mul: float, massive: int = 0, massive_mul: float = 1000.0):
    """Per-channel magnitude c_c and mean shift for LayerNorm inputs."""
    c = np.exp(rng.normal(0.0, sigma_c, size=D))
    n_out = int(round(outlier_frac * D))
    if outlier_frac > 0.0:
        n_out = max(n_out, 1)
    if n_out:
        idx = rng.choice(D, size=n_out, replace=False)
        c[idx] *= outlier_mul
    if massive:
        # fixed positions, spread over the hidden dimension
        pos = (np.arange(massive) * (D // massive) + D // (2 * massive)) % D
        c[pos] = massive_mul
    shift = rng.normal(0.0, 1.0, size=D) * 0.5 * c
    return c, shift


def ln_inputs(rng: np.random.Generator, rows: int, c: np.ndarray, shift: np.ndarray,
              bf16: bool) -> np.ndarray:
    """x[n, ch] = N(0,1) * c[ch] + shift[ch], float32 (on the bf16 grid if `bf16`)."""
    D = c.shape[0]
    x = rng.standard_normal(size=(rows, D), dtype=np.float32)
    x *= c.astype(np.float32)[None, :]
    x += shift.astype(np.float32)[None, :]
    return to_bf16_grid(x) if bf16 else x


def affine_params(rng: np.random.Generator, D: int):
    gamma = rng.normal(1.0, 0.1, size=D).astype(np.float32)
    beta = rng.normal(0.0, 0.1, size=D).astype(np.float32)
    return gamma, beta


def percentile_bounds(a: np.ndarray, axis=None, lo_pct: float = 0.1, hi_pct: float = 99.9):
    """0.1 / 99.9 percentile clipping bounds (the calibration stand-in), float32."""
    lo = np.percentile(a, lo_pct, axis=axis).astype(np.float32)
    hi = np.percentile(a, hi_pct, axis=axis).astype(np.float32)
    # keep the interval non-degenerate and containing zero-width guard
    width = np.maximum(hi - lo, np.float32(1e-6))
    hi = (lo + width).astype(np.float32)
    return lo, hi


def ln_calibration_bounds(x_calib: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float,
                          rms: bool = False):
    """Per-channel bounds of the LayerNorm activation of a calibration batch.

    The normalisation here is PyTorch's library routine, used as a black box to
    shape the input; it is not shared with the oracle or the CUDA path.
    """
    xt = torch.from_numpy(np.ascontiguousarray(x_calib)).double()
    g = torch.from_numpy(gamma).double()
    b = torch.from_numpy(beta).double()
    if rms:
        y = torch.nn.functional.rms_norm(xt, (xt.shape[-1],), weight=g, eps=eps) + b
    else:
        y = torch.nn.functional.layer_norm(xt, (xt.shape[-1],), g, b, eps)
    return percentile_bounds(y.numpy(), axis=0)


def softmax_logits(rng: np.random.Generator, rows: int, L: int) -> np.ndarray:
    """Logits whose Softmax rows are heavy-tailed: top-1 in U(0.3, 0.9), rest ~ k^-alpha."""
    p1 = rng.uniform(0.3, 0.9, size=(rows, 1))
    alpha = rng.uniform(1.0, 2.0, size=(rows, 1))
    if L == 1:
        return rng.normal(0.0, 3.0, size=(rows, 1)).astype(np.float32)
    k = np.arange(1, L, dtype=np.float64)[None, :]
    tail = k ** (-alpha)
    tail *= (1.0 - p1) / tail.sum(axis=1, keepdims=True)
    p = np.concatenate([p1, tail], axis=1)
    # random permutation per row
    order = np.argsort(rng.random(size=(rows, L)), axis=1)
    p = np.take_along_axis(p, order, axis=1)
    logits = np.log(p) + rng.normal(0.0, 3.0, size=(rows, 1))
    return logits.astype(np.float32)


def gemm_codes(rng: np.random.Generator, M: int, N: int, K: int, bits_a: int, bits_w: int):
    """Uniform random activation / weight codes with plausible quantizer parameters."""
    a = rng.integers(0, 1 << bits_a, size=(M, K), dtype=np.int32)
    w = rng.integers(0, 1 << bits_w, size=(N, K), dtype=np.int32)
    s_a = np.float32(rng.uniform(0.01, 0.2))
    z_a = int(rng.integers(0, 1 << bits_a))
    s_w = rng.uniform(0.001, 0.01, size=N).astype(np.float32)
    z_w = rng.integers(0, 1 << bits_w, size=N, dtype=np.int32)
    bias = rng.normal(0.0, 0.02, size=N).astype(np.float32)
    return a, w, s_a, z_a, s_w, z_w, bias
