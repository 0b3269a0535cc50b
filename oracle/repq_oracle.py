"""CPU oracle for the RepQuant inference hot path (arXiv 2402.05628).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what
the hot path computes, written from the paper.  It is used by the tests, by the
smoke check and by the benchmark's CPU-baseline leg; the product path never
calls it.  It shares no code, tables or constants with the CUDA path and does
not import it.

Everything is numpy in float64.  Library primitives used as single steps:
`numpy.matmul` (dense contraction), `numpy.rint` (round half to even),
`numpy.exp`, `numpy.log`, `scipy.special.erf`.  There is no blocking, fusion or
reordering beyond what the cited equations state.

The oracle applies the *complex* quantizers of the quantization process
(channel-wise uniform quantization of LayerNorm activations, log-sqrt2
quantization of Softmax activations); the CUDA path only ever sees the
reparameterized, simple quantizers.  Agreement between the two is therefore a
check of the paper's equivalence claims as well as of the kernels.

Pins (see tests/test_oracle_pins.py): every function below is tied to the
paper's worked example, a closed form, an algebraic identity of Sec. III-C, a
library routine for the un-quantized special case, or brute force on tiny
inputs.  The block composition (`block_forward`, both block forms) is pinned by
a second statement of Eqs. 1-3 and of the quantizer placement written as
explicit per-token / per-head / per-channel loops on tiny blocks, which shares
only the pinned leaf quantizers with it, and is compared with it on the
output, the residual stream and every intermediate code tensor.

Notation follows the paper: s, z quantization scale / zero-point; b bits;
r1 = s / s~, r2 = z - z~; gamma~, beta~, W~, b~ the reparameterized parameters.
Weights are stored [out features j, in features c], i.e. the transpose of the
paper's W in X'W; the paper's "W[:, j]" is row j here.
"""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np
from scipy.special import erf as _erf

F64 = np.float64


# --------------------------------------------------------------------------------------
# Sec. III-A.2  Efficient quantizers
# --------------------------------------------------------------------------------------

def uniform_scale_zero(x_low, x_up, bits: int):
    """Eq. 6: s = (x_up - x_low) / (2^b - 1), z = round(-x_low / s).

    Scales are stored in float32 by every consumer, so s is rounded to float32
    once and z is computed from the stored value.
    """
    x_low = np.asarray(x_low, dtype=F64)
    x_up = np.asarray(x_up, dtype=F64)
    s = (x_up - x_low) / F64(2 ** bits - 1)
    s = s.astype(np.float32).astype(F64)
    z = np.rint(-x_low / s).astype(np.int64)
    return s, z


def quant_uniform(x, s, z, bits: int):
    """Eq. 4: x_q = clip(round(x / s) + z, 0, 2^b - 1).  s, z broadcast against x
    (scalars: layer-wise; length-D vectors: channel-wise, Sec. III-C.1).

    Returns (codes int64, t float64) where t = x / s is the value handed to the
    round operation (used by the tests to recognise rounding near-ties).
    """
    x = np.asarray(x, dtype=F64)
    t = x / np.asarray(s, dtype=F64)
    q = np.rint(t) + np.asarray(z, dtype=F64)
    q = np.clip(q, 0.0, F64(2 ** bits - 1))
    return q.astype(np.int64), t


def dequant_uniform(q, s, z):
    """Eq. 5: x_hat = s (x_q - z)."""
    return np.asarray(s, dtype=F64) * (np.asarray(q, dtype=F64) - np.asarray(z, dtype=F64))


def quant_log2(x, s, bits: int):
    """Eq. 7: x_q = clip(round(-log2(x / s)), 0, 2^b - 1); x = 0 clips to the top code."""
    x = np.asarray(x, dtype=F64)
    with np.errstate(divide="ignore"):
        t = -np.log2(x / F64(s))
    q = np.clip(np.rint(t), 0.0, F64(2 ** bits - 1))
    return q.astype(np.int64), t


def dequant_log2(q, s):
    """Eq. 8: x_hat = s 2^(-x_q)."""
    return F64(s) * np.exp2(-np.asarray(q, dtype=F64))


# --------------------------------------------------------------------------------------
# Sec. III-C.1  LayerNorm activations: channel-wise quantization and its reparameterization
# --------------------------------------------------------------------------------------

def layernorm(X, gamma, beta, eps: float, rms: bool = False):
    """Eq. 9 per token over the D hidden features: (X - E[X]) / sqrt(Var[X] + eps) * gamma + beta,
    population variance.  `rms=True` is the mean-free variant (E[X] := 0, Var := E[X^2])."""
    X = np.asarray(X, dtype=F64)
    if rms:
        mu = np.zeros((X.shape[0], 1), dtype=F64)
    else:
        mu = X.mean(axis=1, keepdims=True)
    d = X - mu
    var = (d * d).mean(axis=1, keepdims=True)
    return d / np.sqrt(var + F64(eps)) * np.asarray(gamma, dtype=F64) + np.asarray(beta, dtype=F64)


def reparam_layernorm(gamma, beta, s, z, W, b) -> Dict[str, np.ndarray]:
    """Eqs. 10-14.  s~ = E[s]; z~ = E[z] rounded to an integer (the paper declares z~ in Z and
    pulls r2 out of the round operation in Eq. 10, which needs integer r2); r1 = s / s~;
    r2 = z - z~; beta~ = (beta + s*r2) / r1; gamma~ = gamma / r1 (Eq. 12);
    W~[j, c] = r1[c] W[j, c]; b~[j] = b[j] - sum_c s[c] r2[c] W[j, c] (Eq. 14)."""
    gamma = np.asarray(gamma, dtype=F64)
    beta = np.asarray(beta, dtype=F64)
    s = np.asarray(s, dtype=F64)
    z = np.asarray(z, dtype=np.int64)
    W = np.asarray(W, dtype=F64)
    b = np.zeros(W.shape[0], dtype=F64) if b is None else np.asarray(b, dtype=F64)
    s_t = s.mean()
    z_t = int(np.rint(z.astype(F64).mean()))
    r1 = s / s_t
    r2 = (z - z_t).astype(F64)
    return dict(s_t=F64(s_t), z_t=z_t, r1=r1, r2=r2,
                gamma_t=gamma / r1, beta_t=(beta + s * r2) / r1,
                W_t=W * r1[None, :], b_t=b - W @ (s * r2))


def quant_weight_rtn(W, bits: int):
    """Channel-wise (per output feature) uniform weight quantization, Eqs. 4-6 with round-to-nearest
    (stand-in for GPTQ, which needs calibration Hessians).  Per row: x_low = min(row, 0),
    x_up = max(row, 0) so that zero is representable and 0 <= z <= 2^b - 1; an all-zero row gets s = 1.
    The scale is rounded to float32 (as stored) before the codes are taken."""
    W = np.asarray(W, dtype=F64)
    lo = np.minimum(W.min(axis=1), 0.0)
    hi = np.maximum(W.max(axis=1), 0.0)
    rng = hi - lo
    s = np.where(rng > 0.0, rng / F64(2 ** bits - 1), 1.0)
    s = s.astype(np.float32).astype(F64)
    z = np.rint(-lo / s).astype(np.int64)
    q, _ = quant_uniform(W, s[:, None], z[:, None], bits)
    return q, s, z


def int_gemm(q, w):
    """acc[n, j] = sum_c q[n, c] w[j, c] in int64 (the integer inner loop of the quantized linear layer)."""
    return np.asarray(q, dtype=np.int64) @ np.asarray(w, dtype=np.int64).T


def linear(x_hat, w_codes, s_w, z_w, b):
    """De-quantized activation times de-quantized weight (Eq. 5 on both operands) plus bias."""
    W_hat = dequant_uniform(w_codes, np.asarray(s_w, dtype=F64)[:, None], np.asarray(z_w)[:, None])
    y = np.asarray(x_hat, dtype=F64) @ W_hat.T
    if b is not None:
        y = y + np.asarray(b, dtype=F64)
    return y


def linear_after_layernorm(q, s, z, rp: Dict[str, np.ndarray], w_codes, s_w, z_w):
    """Right-hand side of Eq. 13 applied to the channel-wise de-quantized LayerNorm activation:
    X^' = s (q - z) per channel (Eq. 5); shifted activation (X^' + s*r2) / r1; times the quantized
    reparameterized weight W~^ = s_w (w - z_w); plus b~ of Eq. 14 (which the paper forms from the
    full-precision W before W~ is quantized)."""
    x_hat = dequant_uniform(q, np.asarray(s, dtype=F64)[None, :], np.asarray(z)[None, :])
    x_shift = (x_hat + (np.asarray(s, dtype=F64) * rp["r2"])[None, :]) / rp["r1"][None, :]
    return linear(x_shift, w_codes, s_w, z_w, rp["b_t"])


# --------------------------------------------------------------------------------------
# Sec. III-C.2  Softmax activations: log-sqrt2 quantizer and its base-2 reparameterization
# --------------------------------------------------------------------------------------

def softmax_rows(S, valid_len: Optional[np.ndarray] = None):
    """Row Softmax of Eq. 3.  `valid_len[i]` (optional) = number of leading keys row i may attend to
    (causal masking is structural: masked keys take no part); masked outputs are returned as 0."""
    S = np.asarray(S, dtype=F64)
    if valid_len is not None:
        cols = np.arange(S.shape[-1])[None, :]
        mask = cols < np.asarray(valid_len)[:, None]
        S = np.where(mask, S, -np.inf)
    m = S.max(axis=-1, keepdims=True)
    e = np.exp(S - m)
    return e / e.sum(axis=-1, keepdims=True)


def quant_logsqrt2(A, s, bits: int):
    """Eq. 15, first line: A_q = clip(round(-log_sqrt2(A / s)), 0, 2^b - 1), the logarithm to base
    sqrt(2) taken as ln(.) / ln(sqrt 2).  A = 0 gives +inf and clips to the top code."""
    A = np.asarray(A, dtype=F64)
    with np.errstate(divide="ignore"):
        t = -np.log(A / F64(s)) / math.log(math.sqrt(2.0))
    q = np.clip(np.rint(t), 0.0, F64(2 ** bits - 1))
    return q.astype(np.int64), t


def quant_logsqrt2_base2(A, s, bits: int):
    """Eq. 15, second line: the same codes through -2 log2(A / s)."""
    A = np.asarray(A, dtype=F64)
    with np.errstate(divide="ignore"):
        t = -2.0 * np.log2(A / F64(s))
    q = np.clip(np.rint(t), 0.0, F64(2 ** bits - 1))
    return q.astype(np.int64), t


def dequant_logsqrt2(q, s):
    """Eq. 16, first line: A^ = s sqrt(2)^(-A_q) = s 2^(-A_q / 2) (evaluated in the base-2 form, whose
    base is exact in binary floating point)."""
    return F64(s) * np.exp2(-np.asarray(q, dtype=F64) / 2.0)


def dequant_log2_reparam(q, s):
    """Eq. 16, last line, with Eq. 17: A^ = s~ 2^floor(-A_q / 2), s~ = s [1(A_q)(sqrt2 - 1) + 1],
    1(.) the parity indicator."""
    q = np.asarray(q, dtype=np.int64)
    parity = (q % 2).astype(F64)
    s_t = F64(s) * (parity * (math.sqrt(2.0) - 1.0) + 1.0)
    return s_t * np.exp2(np.floor(-q.astype(F64) / 2.0))


# --------------------------------------------------------------------------------------
# Sec. III-D  Per-channel dual clipping (Eqs. 18-20)
# --------------------------------------------------------------------------------------

def dual_clip_bounds(x_max, x_min, alpha1, alpha2):
    """Eqs. 18-19: X'_up = max_d * Sigmoid(alpha1), X'_low = min_d * Sigmoid(alpha2), per channel."""
    sig = lambda a: 1.0 / (1.0 + np.exp(-np.asarray(a, dtype=F64)))
    return np.asarray(x_max, dtype=F64) * sig(alpha1), np.asarray(x_min, dtype=F64) * sig(alpha2)


def dual_clip_loss_grad(X, alpha1, alpha2, bits: int):
    """Objective of Eq. 20 per channel, ||X'_{:,d} - X^'_{:,d}||^2 with the channel-wise quantizer of Eqs. 4-6 built
    on the bounds of Eqs. 18-19, and its gradient with respect to (alpha1, alpha2).

    The round operations (of x/s in Eq. 4 and of -x_low/s in Eq. 6) are passed straight through in the backward
    direction (derivative 1), the clip passes the gradient on [0, 2^b - 1] inclusive and blocks it outside; the
    paper learns the factors by gradient descent (Sec. IV-A) without printing these conventions, which are the
    usual ones for learned quantizer bounds.  With u = x/s, zc = -x_low/s, r = round(u), z = round(zc),
    q = clip(r + z, 0, Q), Q = 2^b - 1 and x^ = s (q - z):
        inside the clip   dx^/ds = r - u            dx^/dx_low (s fixed) = 0
        clipped           dx^/ds = q - z + zc       dx^/dx_low (s fixed) = 1
    and s = (x_up - x_low) / Q, x_up = max * sig(alpha1), x_low = min * sig(alpha2).
    Returns (loss[D], dloss/dalpha1[D], dloss/dalpha2[D])."""
    X = np.asarray(X, dtype=F64)
    Q = F64(2 ** bits - 1)
    x_max, x_min = X.max(axis=0), X.min(axis=0)
    sg1 = 1.0 / (1.0 + np.exp(-np.asarray(alpha1, dtype=F64)))
    sg2 = 1.0 / (1.0 + np.exp(-np.asarray(alpha2, dtype=F64)))
    up, low = x_max * sg1, x_min * sg2
    s = (up - low) / Q
    u = X / s
    zc = -low / s
    r, z = np.rint(u), np.rint(zc)
    pre = r + z
    q = np.clip(pre, 0.0, Q)
    x_hat = s * (q - z)
    inside = (pre >= 0.0) & (pre <= Q)
    g = 2.0 * (x_hat - X)                                   # dL/dx^
    dxh_ds = np.where(inside, r - u, q - z + zc)
    dxh_dlow = np.where(inside, 0.0, 1.0)
    dL_ds = (g * dxh_ds).sum(axis=0)
    dL_dlow_direct = (g * dxh_dlow).sum(axis=0)
    dL_dup = dL_ds / Q
    dL_dlow = dL_dlow_direct - dL_ds / Q
    loss = ((x_hat - X) ** 2).sum(axis=0)
    return loss, dL_dup * x_max * sg1 * (1.0 - sg1), dL_dlow * x_min * sg2 * (1.0 - sg2)


def dual_clip(X, bits: int, iters: int = 100, lr: float = 0.01, alpha0: float = 0.0,
              beta1: float = 0.9, beta2: float = 0.999, adam_eps: float = 1e-8):
    """Per-channel dual clipping (Sec. III-D): Adam (Sec. IV-A: 100 iterations, learning rate 0.01; the moment
    decay rates and epsilon are the optimizer's customary defaults, which the paper does not restate) on the
    clipping factors of every channel of the LayerNorm activations X [tokens, D], objective of Eq. 20.
    `alpha0` is the factors' initial value, which the paper does not give (0: the bounds start at half of each
    channel's extremes; 2: at 0.88 of them, from where 100 steps of 0.01 reach contractions of 0.73 to 0.95).  Returns dict(x_low, x_up, alpha1, alpha2, loss0, loss) with loss0 / loss the per-channel
    objective before the first and after the last update."""
    X = np.asarray(X, dtype=F64)
    D = X.shape[1]
    a1 = np.full(D, alpha0, dtype=F64)
    a2 = np.full(D, alpha0, dtype=F64)
    m1, v1, m2, v2 = (np.zeros(D, dtype=F64) for _ in range(4))
    loss0 = None
    for t in range(1, iters + 1):
        loss, g1, g2 = dual_clip_loss_grad(X, a1, a2, bits)
        if loss0 is None:
            loss0 = loss
        m1 = beta1 * m1 + (1.0 - beta1) * g1
        v1 = beta2 * v1 + (1.0 - beta2) * g1 * g1
        m2 = beta1 * m2 + (1.0 - beta1) * g2
        v2 = beta2 * v2 + (1.0 - beta2) * g2 * g2
        c1, c2 = 1.0 - beta1 ** t, 1.0 - beta2 ** t
        a1 = a1 - lr * (m1 / c1) / (np.sqrt(v1 / c2) + adam_eps)
        a2 = a2 - lr * (m2 / c1) / (np.sqrt(v2 / c2) + adam_eps)
    loss, _, _ = dual_clip_loss_grad(X, a1, a2, bits)
    up, low = dual_clip_bounds(X.max(axis=0), X.min(axis=0), a1, a2)
    return dict(x_low=low, x_up=up, alpha1=a1, alpha2=a2, loss0=loss if loss0 is None else loss0, loss=loss)


# --------------------------------------------------------------------------------------
# Sec. III-A.1  Transformer block (Eqs. 1-3)
# --------------------------------------------------------------------------------------

def gelu(x):
    """GELU, exact erf form."""
    x = np.asarray(x, dtype=F64)
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def round_bf16(x):
    """Round-to-nearest-even onto the bf16 grid (8 significant bits), straight from float64
    (models a bf16-stored activation tensor; sub-normal and overflow ranges are not modelled)."""
    x = np.asarray(x, dtype=F64)
    m, e = np.frexp(x)                      # x = m 2^e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0) / 256.0, e)


def silu(x):
    """SiLU, x sigmoid(x): the gate non-linearity of the LLaMA-style MLP (not in the paper's block; see
    `block_forward`)."""
    x = np.asarray(x, dtype=F64)
    return x / (1.0 + np.exp(-x))


def rope(X, B: int, L: int, H: int, base: float = 10000.0):
    """Rotary position embedding on a [B*L, D] matrix of H heads (not in the paper's block; the LLaMA models of
    Sec. IV-A apply it to Q and K).  Within a head of d_h channels, the consecutive pair (2i, 2i+1) of the token
    at position m is one complex number, multiplied by exp(j m theta_i), theta_i = base^(-2i / d_h):
        x'[2i]   = x[2i] cos(m theta_i) - x[2i+1] sin(m theta_i)
        x'[2i+1] = x[2i] sin(m theta_i) + x[2i+1] cos(m theta_i)."""
    X = np.asarray(X, dtype=F64)
    M, D = X.shape
    dh = D // H
    theta = F64(base) ** (-np.arange(0, dh, 2, dtype=F64) / F64(dh))       # [dh/2]
    ang = np.arange(L, dtype=F64)[:, None] * theta[None, :]                 # [L, dh/2]
    cos = np.tile(np.cos(ang), (B, H))                                      # [B*L, D/2]
    sin = np.tile(np.sin(ang), (B, H))
    even, odd = X[:, 0::2], X[:, 1::2]
    out = np.empty_like(X)
    out[:, 0::2] = even * cos - odd * sin
    out[:, 1::2] = even * sin + odd * cos
    return out


def attention(Qc, Kc, Vc, qp: dict, B: int, L: int, H: int, softmax_s: float, bits_p: int,
              causal: bool, keep: bool = False):
    """Eq. 3 per (batch, head) on de-quantized Q, K, V, with the Softmax output passed through the
    log-sqrt2 quantizer (Eq. 15) and de-quantized by Eq. 16's first line.
    Qc/Kc/Vc: [B*L, D] integer codes; qp: layer-wise (s, z) of q, k, v.  The scale is 1/sqrt(d_h)
    (per-head feature size).  Returns O [B*L, D] and, if `keep`, scores / codes per (b, h)."""
    M, D = Qc.shape
    dh = D // H
    Qh = dequant_uniform(Qc, qp["s_q"], qp["z_q"])
    Kh = dequant_uniform(Kc, qp["s_k"], qp["z_k"])
    Vh = dequant_uniform(Vc, qp["s_v"], qp["z_v"])
    O = np.empty((M, D), dtype=F64)
    kept = dict(S=[], p=[], t=[]) if keep else None
    valid = (np.arange(L) + 1) if causal else None
    for bi in range(B):
        r = slice(bi * L, (bi + 1) * L)
        for h in range(H):
            c = slice(h * dh, (h + 1) * dh)
            S = Qh[r, c] @ Kh[r, c].T / math.sqrt(dh)
            A = softmax_rows(S, valid)
            p, t = quant_logsqrt2(A, softmax_s, bits_p)
            A_hat = dequant_logsqrt2(p, softmax_s)
            if causal:
                A_hat = np.where(np.arange(L)[None, :] < valid[:, None], A_hat, 0.0)
            O[r, c] = A_hat @ Vh[r, c]
            if keep:
                kept["S"].append(S)
                kept["p"].append(p)
                kept["t"].append(t)
    return O, kept


def percentile_bounds(v, lo_pct: float = 0.1, hi_pct: float = 99.9):
    """Percentile calibration of a layer-wise quantizer (Sec. IV-A names the strategy, not the percentiles; the
    workloads fix 0.1 / 99.9): the bounds handed to Eq. 6, rounded to float32 as they are stored."""
    lo, hi = np.percentile(np.asarray(v, dtype=F64), [lo_pct, hi_pct])
    return np.float32(lo), np.float32(hi)


def block_forward(w, keep: bool = False, calibrate: Optional[dict] = None) -> Dict[str, np.ndarray]:
    """Eqs. 1-2 with every matrix-multiplication input quantized (Sec. III-A.1, IV-A):
    X_bar = MSA(LN(X)) + X,  Y = MLP(LN(X_bar)) + X_bar.

    `w` is a workload (workloads.BlockInputs): full-precision parameters plus clipping bounds.
    LayerNorm activations: channel-wise quantization (s, z per channel from Eq. 6).  Softmax:
    log-sqrt2.  Every other activation: layer-wise uniform.  Weights: channel-wise RTN; the weights
    that follow a LayerNorm are the reparameterized W~ (rounded to float32, as stored).
    With bf16 activations the residual stream X_bar is stored in bf16.

    Two block forms.  The default is the paper's own block (LayerNorm, MLP = fc2(GELU(fc1(.)))).  The paper also
    evaluates LLaMA models (Sec. IV-A) but never writes their block down; `cfg["arch"] == "llama"` selects that
    form, with the same quantizer placement (every matrix-multiplication input quantized): the normalisation is
    the mean-free one (RMSNorm: Eq. 9 with E[X] := 0, Var := E[X^2]; its channel-wise quantizer is reparameterized
    by Eqs. 10-14 all the same, beta being whatever the workload holds, zero for RMSNorm), rotary position
    embedding is applied to the full-precision Q and K of the projection before their quantizers, and the MLP is
    down(SiLU(gate(.)) * up(.)) with `w_fc1` = [gate; up] stacked on the output axis, the product being the
    quantized input of the down projection `w_fc2`.

    `calibrate` (a dict, possibly empty) turns the pass into the sequential pipeline of Algorithm 1 on a
    calibration batch `w.x`, with round-to-nearest in GPTQ's place: every quantizer's bounds are found on the input
    that reaches it through the layers already quantized (Algorithm 1 collects each layer's input in one
    traversal) instead of being taken from `w`: per-channel dual clipping (Eqs. 18-20; keys `alpha0`, `iters`,
    `lr`) for the two LayerNorm activations, percentile calibration (keys `lo_pct`, `hi_pct`) for the layer-wise
    quantizers.  The bounds found are returned under "bounds", "ln1_lo", "ln1_hi", "ln2_lo", "ln2_hi".
    """
    cfg = w.cfg
    B, L, D, H = cfg["B"], cfg["L"], cfg["D"], cfg["H"]
    ba, bw, bp = cfg["bits_a"], cfg["bits_w"], cfg["bits_p"]
    out: Dict[str, np.ndarray] = {}
    x = np.asarray(w.x, dtype=F64)

    llama = cfg.get("arch", "vit") == "llama"
    cal = calibrate
    found: Dict[str, tuple] = {}

    def post_ln_linear(X_in, gamma, beta, lo, hi, W, b, tag):
        X1 = layernorm(X_in, gamma, beta, cfg["eps"], rms=llama)
        if cal is not None:
            # the activations as the calibration tool holds them (float32), then Eqs. 18-20
            X1_32 = X1.astype(np.float32).astype(F64)
            r = dual_clip(X1_32, ba, iters=cal.get("iters", 100), lr=cal.get("lr", 0.01), alpha0=cal.get("alpha0", 0.0))
            lo, hi = r["x_low"].astype(np.float32), r["x_up"].astype(np.float32)
            out[tag + "_lo"], out[tag + "_hi"] = lo, hi
        s, z = uniform_scale_zero(lo, hi, ba)
        q, t = quant_uniform(X1, s[None, :], z[None, :], ba)            # channel-wise
        rp = reparam_layernorm(gamma, beta, s, z, W, b)
        W_t32 = rp["W_t"].astype(np.float32).astype(F64)
        wc, s_w, z_w = quant_weight_rtn(W_t32, bw)
        y = linear_after_layernorm(q, s, z, rp, wc, s_w, z_w)
        if keep:
            out[tag + "_codes"], out[tag + "_t"] = q, t
            out[tag + "_s"], out[tag + "_z"] = s, z
            out[tag + "_rp"], out[tag + "_wcodes"] = rp, wc
            out[tag + "_sw"], out[tag + "_zw"] = s_w, z_w
        return y

    def requant(v, name):
        if cal is not None:
            found[name] = percentile_bounds(v, cal.get("lo_pct", 0.1), cal.get("hi_pct", 99.9))
            lo, hi = found[name]
        else:
            lo, hi = w.bounds[name]
        s, z = uniform_scale_zero(lo, hi, ba)
        q, t = quant_uniform(v, s, z, ba)
        if keep:
            out[name + "_codes"], out[name + "_t"] = q, t
        return q, float(s), int(z)

    qkv = post_ln_linear(x, w.ln1_gamma, w.ln1_beta, w.ln1_lo, w.ln1_hi, w.w_qkv, w.b_qkv, "ln1")
    Q_fp, K_fp = qkv[:, :D], qkv[:, D:2 * D]
    if llama:
        Q_fp = rope(Q_fp, B, L, H, cfg.get("rope_base", 10000.0))
        K_fp = rope(K_fp, B, L, H, cfg.get("rope_base", 10000.0))
    Qc, s_q, z_q = requant(Q_fp, "q")
    Kc, s_k, z_k = requant(K_fp, "k")
    Vc, s_v, z_v = requant(qkv[:, 2 * D:], "v")
    qp = dict(s_q=s_q, z_q=z_q, s_k=s_k, z_k=z_k, s_v=s_v, z_v=z_v)
    O, kept = attention(Qc, Kc, Vc, qp, B, L, H, w.softmax_scale, bp, cfg["causal"], keep)
    if keep:
        out["scores"], out["p_codes"], out["p_t"] = kept["S"], kept["p"], kept["t"]
        out["attn_pre"] = O
    Oc, s_o, z_o = requant(O, "attn")
    wc, s_w, z_w = quant_weight_rtn(w.w_proj, bw)
    x_bar = linear(dequant_uniform(Oc, s_o, z_o), wc, s_w, z_w, w.b_proj) + x
    if cfg["act"] == "bf16":
        x_bar = round_bf16(x_bar)
    if keep:
        out["x_bar"] = x_bar

    h_pre = post_ln_linear(x_bar, w.ln2_gamma, w.ln2_beta, w.ln2_lo, w.ln2_hi, w.w_fc1, w.b_fc1, "ln2")
    if llama:
        n_mlp = cfg["MLP"]
        h_act = silu(h_pre[:, :n_mlp]) * h_pre[:, n_mlp:]
    else:
        h_act = gelu(h_pre)
    hc, s_h, z_h = requant(h_act, "hidden")
    wc, s_w, z_w = quant_weight_rtn(w.w_fc2, bw)
    out["y"] = linear(dequant_uniform(hc, s_h, z_h), wc, s_w, z_w, w.b_fc2) + x_bar
    if cal is not None:
        out["bounds"] = found
    return out
