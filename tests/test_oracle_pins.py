"""Pins for the CPU oracle: each oracle function is checked against something other than itself —
the paper's worked example, closed forms, algebraic identities of Sec. III-C, library routines for
un-quantized special cases, or brute force on tiny inputs.  No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import repq_oracle as orc
from workloads import make_block_inputs


# ------------------------------------------------------------------ worked example (golden fixture)

def _read_golden(path):
    rows = []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        kind, a, code, deq = line.split()
        rows.append((kind, float(a), int(code), float(deq)))
    return rows


def test_log_quantizer_worked_example(golden_dir):
    rows = _read_golden(os.path.join(golden_dir, "log_quantizer_example.txt"))
    assert len(rows) >= 10
    for kind, a, code, deq in rows:
        if kind == "log2":
            q, _ = orc.quant_log2(np.array([a]), 1.0, 4)
            d = orc.dequant_log2(q, 1.0)
        else:
            q, _ = orc.quant_logsqrt2(np.array([a]), 1.0, 4)
            d = orc.dequant_logsqrt2(q, 1.0)
        assert int(q[0]) == code, (kind, a)
        assert abs(float(d[0]) - deq) < 1e-15, (kind, a)
    # interval ends printed by the paper: the open interval between them maps to code 1
    grid = np.linspace(math.sqrt(2) ** -1.5, math.sqrt(2) ** -0.5, 1001)[1:-1]
    assert np.all(orc.quant_logsqrt2(grid, 1.0, 4)[0] == 1)
    grid = np.linspace(2 ** -1.5, 2 ** -0.5, 1001)[1:-1]
    assert np.all(orc.quant_log2(grid, 1.0, 4)[0] == 1)


# ------------------------------------------------------------------ uniform quantizer (Eqs. 4-6)

def test_uniform_hand_values():
    # x_low = -1, x_up = 2, b = 4: s = 3/15 = 0.2 (float32-rounded), z = round(5) = 5
    s, z = orc.uniform_scale_zero(-1.0, 2.0, 4)
    assert abs(float(s) - 0.2) < 1e-8 and int(z) == 5
    # exact binary scale so that ties are real ties: s = 0.25, z = 3
    q, t = orc.quant_uniform(np.array([0.625, 0.875, -0.125, 100.0, -100.0, 0.3]), 0.25, 3, 4)
    # 0.625/0.25 = 2.5 -> 2 (half to even) + 3 = 5 ; 0.875/0.25 = 3.5 -> 4 + 3 = 7 ; -0.5 -> -0 + 3 = 3
    assert q.tolist() == [5, 7, 3, 15, 0, 4]
    assert np.allclose(orc.dequant_uniform(q, 0.25, 3), [0.5, 1.0, 0.0, 3.0, -0.75, 0.25])
    # round first, then add z, then clip: with z = 20 > 2^b - 1 a small x still clips to 15
    assert orc.quant_uniform(np.array([0.0]), 0.25, 20, 4)[0].tolist() == [15]


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_uniform_grid_properties(bits):
    rng = np.random.default_rng(5)
    lo, hi = -1.7, 3.1
    s, z = orc.uniform_scale_zero(lo, hi, bits)
    x = np.sort(rng.uniform(lo, hi, 20001))
    q, _ = orc.quant_uniform(x, s, z, bits)
    assert q.min() >= 0 and q.max() <= 2 ** bits - 1
    assert np.all(np.diff(q) >= 0)                                   # monotone
    # the representable grid s (k - z) covers [lo, hi] up to half a step at each end (z is rounded)
    inside = (x >= float(s) * (0 - z)) & (x <= float(s) * (2 ** bits - 1 - z))
    err = np.abs(orc.dequant_uniform(q, s, z) - x)
    assert err[inside].max() <= float(s) / 2 * (1 + 1e-12)
    assert abs(int(orc.quant_uniform(np.array([lo]), s, z, bits)[0][0]) - 0) <= 1
    assert abs(int(orc.quant_uniform(np.array([hi]), s, z, bits)[0][0]) - (2 ** bits - 1)) <= 1
    # every code is hit and dequantization of code k is s (k - z)
    assert len(np.unique(q)) == 2 ** bits
    k = np.arange(2 ** bits)
    assert np.array_equal(orc.quant_uniform(orc.dequant_uniform(k, s, z), s, z, bits)[0], k)


# ------------------------------------------------------------------ LayerNorm (Eq. 9)

def test_layernorm_matches_library():
    rng = np.random.default_rng(1)
    X = rng.normal(size=(37, 96)) * rng.lognormal(size=96) + rng.normal(size=96)
    g, b = rng.normal(1, 0.1, 96), rng.normal(0, 0.1, 96)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(X), (96,), torch.from_numpy(g),
                                         torch.from_numpy(b), 1e-6).numpy()
    assert np.abs(orc.layernorm(X, g, b, 1e-6) - ref).max() < 1e-12
    # closed form on one row: x = [1, 2, 3, 6]: mean 3, population variance 3.5
    y = orc.layernorm(np.array([[1.0, 2.0, 3.0, 6.0]]), np.ones(4), np.zeros(4), 0.0)
    assert np.allclose(y[0], (np.array([1, 2, 3, 6]) - 3) / math.sqrt(3.5), atol=1e-15)
    # mean-free variant: x / sqrt(mean x^2)
    y = orc.layernorm(np.array([[3.0, 4.0]]), np.ones(2), np.zeros(2), 0.0, rms=True)
    assert np.allclose(y[0], np.array([3.0, 4.0]) / math.sqrt(12.5), atol=1e-15)


# ------------------------------------------------------------------ reparameterization (Eqs. 10-14)

def _ln_case(seed=3, n=64, D=48, N=20, bits=4):
    rng = np.random.default_rng(seed)
    X = rng.normal(size=(n, D)) * rng.lognormal(0, 1.0, size=D) + rng.normal(size=D)
    g, b = rng.normal(1, 0.1, D), rng.normal(0, 0.1, D)
    X1 = orc.layernorm(X, g, b, 1e-6)
    s, z = orc.uniform_scale_zero(np.percentile(X1, 1, axis=0), np.percentile(X1, 99, axis=0), bits)
    W = rng.normal(0, 0.02, size=(N, D))
    bias = rng.normal(0, 0.02, size=N)
    return X, g, b, X1, s, z, W, bias


def test_reparam_identities():
    X, g, b, X1, s, z, W, bias = _ln_case()
    rp = orc.reparam_layernorm(g, b, s, z, W, bias)
    assert isinstance(rp["z_t"], int)
    assert np.all(rp["r2"] == np.rint(rp["r2"]))                       # r2 integer
    assert np.allclose(s / rp["r1"], rp["s_t"], rtol=1e-15)            # Eq. 11: s~ = s / r1
    assert np.array_equal(z - rp["r2"], np.full_like(z, rp["z_t"], dtype=float))   # Eq. 10: z~ = z - r2
    assert abs(rp["s_t"] - s.mean()) < 1e-18 and abs(rp["z_t"] - z.mean()) <= 0.5
    # Eq. 12 produces the shifted activation (X' + s*r2) / r1
    X1t = orc.layernorm(X, rp["gamma_t"], rp["beta_t"], 1e-6)
    assert np.abs(X1t - (X1 + s * rp["r2"]) / rp["r1"]).max() < 1e-10
    # Eq. 13: X'W + b = X~'W~ + b~
    lhs = X1 @ W.T + bias
    rhs = X1t @ rp["W_t"].T + rp["b_t"]
    assert np.abs(lhs - rhs).max() < 1e-11 * max(1.0, np.abs(lhs).max())
    # Eq. 14 written out with loops on a corner
    j = 3
    assert abs(rp["b_t"][j] - (bias[j] - sum(s[c] * rp["r2"][c] * W[j, c] for c in range(len(s))))) < 1e-14
    assert np.allclose(rp["W_t"][j], rp["r1"] * W[j], rtol=1e-15)


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_codes_fixed_under_reparam(bits):
    """'The quantized integer values of LayerNorm activations are fixed' (end of Sec. III-C.1):
    channel-wise codes on X' equal layer-wise codes on X~'; differences only at rounding near-ties."""
    X, g, b, X1, s, z, W, bias = _ln_case(seed=7, n=512, D=96, bits=bits)
    rp = orc.reparam_layernorm(g, b, s, z, W, bias)
    q_cw, t_cw = orc.quant_uniform(X1, s[None, :], z[None, :], bits)
    X1t = orc.layernorm(X, rp["gamma_t"], rp["beta_t"], 1e-6)
    q_lw, t_lw = orc.quant_uniform(X1t, rp["s_t"], rp["z_t"], bits)
    diff = q_cw != q_lw
    frac_part = np.abs(t_cw - np.floor(t_cw) - 0.5)
    assert np.all(frac_part[diff] < 1e-9)          # any mismatch sits on a tie (to fp64 round-off)
    assert diff.sum() <= 2
    # the pre-rounding values differ by exactly r2 (integer), which is why the codes coincide
    assert np.abs((t_lw - t_cw) - rp["r2"][None, :]).max() < 1e-9
    # and the de-quantized values are related by the shift: s~ (q - z~) = (s (q - z) + s r2) / r1
    lhs = orc.dequant_uniform(q_cw, rp["s_t"], rp["z_t"])
    rhs = (orc.dequant_uniform(q_cw, s[None, :], z[None, :]) + s * rp["r2"]) / rp["r1"]
    assert np.abs(lhs - rhs).max() < 1e-12


def test_reparam_trivial_case_is_plain_layerwise():
    """r1 = 1, r2 = 0 (all channels share s, z) leaves every parameter untouched."""
    rng = np.random.default_rng(2)
    D, N = 16, 5
    g, b = rng.normal(1, 0.1, D), rng.normal(0, 0.1, D)
    W, bias = rng.normal(size=(N, D)), rng.normal(size=N)
    rp = orc.reparam_layernorm(g, b, np.full(D, 0.125), np.full(D, 7), W, bias)
    assert rp["s_t"] == 0.125 and rp["z_t"] == 7
    for a, ref in ((rp["gamma_t"], g), (rp["beta_t"], b), (rp["W_t"], W), (rp["b_t"], bias)):
        assert np.array_equal(a, ref)


def test_linear_after_layernorm_equals_layerwise_form():
    """Eq. 13's right-hand side on de-quantized codes equals s~ (q - z~) W~^ + b~, the form the
    integer GEMM evaluates; checked with explicit integer loops on a corner."""
    X, g, b, X1, s, z, W, bias = _ln_case(seed=11, n=9, D=24, N=6)
    rp = orc.reparam_layernorm(g, b, s, z, W, bias)
    q, _ = orc.quant_uniform(X1, s[None, :], z[None, :], 4)
    wc, s_w, z_w = orc.quant_weight_rtn(rp["W_t"], 4)
    y = orc.linear_after_layernorm(q, s, z, rp, wc, s_w, z_w)
    for n, j in ((0, 0), (4, 3), (8, 5)):
        corr = sum((int(q[n, c]) - rp["z_t"]) * (int(wc[j, c]) - int(z_w[j])) for c in range(24))
        ref = float(rp["s_t"]) * float(s_w[j]) * corr + rp["b_t"][j]
        assert abs(y[n, j] - ref) < 1e-12 * max(1.0, abs(ref))
    # four-term expansion of the zero-point correction, all integers
    acc = orc.int_gemm(q, wc)
    asum, wsum = q.sum(axis=1), wc.sum(axis=1)
    corr = acc - z_w[None, :] * asum[:, None] - rp["z_t"] * wsum[None, :] + 24 * rp["z_t"] * z_w[None, :]
    ref = float(rp["s_t"]) * s_w[None, :] * corr + rp["b_t"][None, :]
    assert np.abs(y - ref).max() < 1e-12 * np.abs(ref).max()


# ------------------------------------------------------------------ weights, integer GEMM, linear

@pytest.mark.parametrize("bits", [4, 6, 8])
def test_weight_rtn(bits):
    rng = np.random.default_rng(bits)
    W = rng.normal(0, 0.02, size=(13, 40))
    W[5] = 0.0                    # degenerate row
    W[6] = np.abs(W[6])           # one-sided row
    q, s, z = orc.quant_weight_rtn(W, bits)
    qmax = 2 ** bits - 1
    assert q.min() >= 0 and q.max() <= qmax and z.min() >= 0 and z.max() <= qmax
    W_hat = orc.dequant_uniform(q, s[:, None], z[:, None])
    assert np.all(np.abs(W_hat - W) <= s[:, None] * 0.5 * (1 + 1e-6) + 1e-12)
    assert np.all(W_hat[5] == 0.0) and z[6] == 0
    # a value of exactly zero is reproduced exactly
    W2 = W.copy()
    W2[:, 0] = 0.0
    q2, s2, z2 = orc.quant_weight_rtn(W2, bits)
    assert np.all(orc.dequant_uniform(q2[:, 0], s2, z2) == 0.0)
    # scale is the float32 rounding of range / (2^b - 1)
    r = np.maximum(W.max(1), 0) - np.minimum(W.min(1), 0)
    assert np.array_equal(s[[0, 1, 2]], (r / qmax).astype(np.float32).astype(np.float64)[[0, 1, 2]])


def test_int_gemm_brute_force():
    rng = np.random.default_rng(0)
    M, N, K = 7, 5, 19
    a = rng.integers(0, 256, size=(M, K))
    w = rng.integers(0, 256, size=(N, K))
    acc = orc.int_gemm(a, w)
    assert acc.dtype == np.int64
    for m in range(M):
        for n in range(N):
            assert acc[m, n] == sum(int(a[m, k]) * int(w[n, k]) for k in range(K))


def test_linear_brute_force():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(3, 8))
    wc = rng.integers(0, 16, size=(4, 8))
    s_w, z_w, b = rng.uniform(0.01, 0.1, 4), rng.integers(0, 16, 4), rng.normal(size=4)
    y = orc.linear(x, wc, s_w, z_w, b)
    for n in range(3):
        for j in range(4):
            ref = sum(x[n, c] * s_w[j] * (int(wc[j, c]) - int(z_w[j])) for c in range(8)) + b[j]
            assert abs(y[n, j] - ref) < 1e-13


# ------------------------------------------------------------------ Softmax and the log quantizers

def test_softmax_properties():
    from scipy.special import softmax as sp_softmax
    rng = np.random.default_rng(9)
    S = rng.normal(0, 5, size=(33, 57))
    A = orc.softmax_rows(S)
    assert np.abs(A.sum(axis=1) - 1).max() < 1e-14
    assert np.abs(A - orc.softmax_rows(S + 123.456)).max() < 1e-13
    assert np.abs(A - sp_softmax(S, axis=1)).max() < 1e-15
    # causal: row i sees keys 0..i only
    Sq = rng.normal(size=(6, 6))
    Ac = orc.softmax_rows(Sq, np.arange(6) + 1)
    for i in range(6):
        assert np.abs(Ac[i, : i + 1] - sp_softmax(Sq[i, : i + 1])).max() < 1e-15
        assert np.all(Ac[i, i + 1:] == 0.0)
    assert Ac[0, 0] == 1.0


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_logsqrt2_dequant_identity_all_codes(bits):
    """Eq. 16: s sqrt2^-q equals s~ 2^floor(-q/2) for every code (the reparameterization is exact)."""
    q = np.arange(2 ** bits)
    for s in (1.0, 0.7, 0.3183):
        a = orc.dequant_logsqrt2(q, s)
        r = orc.dequant_log2_reparam(q, s)
        even = q % 2 == 0
        assert np.array_equal(a[even], r[even])
        assert np.abs(a[~even] - r[~even]).max() <= 4 * np.finfo(np.float64).eps * s
        # explicit cases of Eq. 16: even q -> s 2^(-q/2); odd q -> s 2^(-(q+1)/2) sqrt2
        for k in (0, 1, 2, 3, 2 ** bits - 2, 2 ** bits - 1):
            ref = s * 2.0 ** (-k // 2 if k % 2 == 0 else -(k + 1) // 2) * (1.0 if k % 2 == 0 else math.sqrt(2))
            assert abs(r[k] - ref) <= 2 * np.finfo(np.float64).eps * ref
        # even codes of the log-sqrt2 quantizer are the plain log2 quantizer's levels (Eq. 8)
        assert np.array_equal(a[even], orc.dequant_log2(q[even] // 2, s))


@pytest.mark.parametrize("bits", [4, 8])
def test_logsqrt2_quant_forms_agree(bits):
    """Eq. 15: the base-sqrt2 form and the -2 log2 form give the same codes; codes fall as A grows;
    the reconstruction error in the log domain is at most half a level."""
    rng = np.random.default_rng(17)
    A = np.concatenate([rng.uniform(0, 1, 5000), 10.0 ** rng.uniform(-12, 0, 5000), [0.0, 1.0]])
    for s in (1.0, 0.7):
        q1, t1 = orc.quant_logsqrt2(A, s, bits)
        q2, t2 = orc.quant_logsqrt2_base2(A, s, bits)
        with np.errstate(invalid="ignore"):
            near_tie = np.abs(t1 - np.floor(t1) - 0.5) < 1e-9
        assert np.array_equal(q1[~near_tie], q2[~near_tie])
        order = np.argsort(A)
        assert np.all(np.diff(q1[order]) <= 0)
        assert q1[-2] == 2 ** bits - 1                       # A = 0 clips to the top code
        assert q1[-1] == 0                                   # A >= s: non-positive level clips to 0
        un = (q1 > 0) & (q1 < 2 ** bits - 1)
        rec = orc.dequant_logsqrt2(q1, s)
        assert np.abs(np.log2(rec[un] / A[un])).max() <= 0.25 + 1e-12
    # s = 0.7: A = 0.5 -> -2 log2(0.714) = 0.97 -> 1 ; A = 0.7 -> 0
    assert orc.quant_logsqrt2(np.array([0.5, 0.7]), 0.7, 4)[0].tolist() == [1, 0]
    # s = 0.7: A = 0.5 -> -2 log2(0.714) = 0.97 -> 1 ; A = 0.7 -> 0
    assert orc.quant_logsqrt2(np.array([0.5, 0.7]), 0.7, 4)[0].tolist() == [1, 0]
    # hand values, s = 1: A = 2^-3 -> 6 ; 2^-3.5 -> 7 ; 0.3 -> round(3.474) = 3
    assert orc.quant_logsqrt2(np.array([0.125, 2 ** -3.5 * 1.0001, 0.3]), 1.0, 4)[0].tolist() == [6, 7, 3]


def test_attention_brute_force():
    rng = np.random.default_rng(21)
    B, L, H, dh = 2, 5, 2, 4
    D = H * dh
    Qc, Kc, Vc = (rng.integers(0, 16, size=(B * L, D)) for _ in range(3))
    qp = dict(s_q=0.3, z_q=7, s_k=0.2, z_k=8, s_v=0.1, z_v=6)
    for causal in (False, True):
        O, _ = orc.attention(Qc, Kc, Vc, qp, B, L, H, 1.0, 4, causal)
        for b in range(B):
            for h in range(H):
                for i in range(L):
                    keys = range(i + 1) if causal else range(L)
                    sc = [sum(0.3 * (Qc[b * L + i, h * dh + d] - 7) * 0.2 * (Kc[b * L + j, h * dh + d] - 8)
                              for d in range(dh)) / math.sqrt(dh) for j in keys]
                    m = max(sc)
                    e = [math.exp(v - m) for v in sc]
                    a = [v / sum(e) for v in e]
                    codes = [min(15, max(0, int(np.rint(-2 * math.log2(v))))) if v > 0 else 15 for v in a]
                    for d in range(dh):
                        ref = sum(2.0 ** (-c / 2) * 0.1 * (Vc[b * L + j, h * dh + d] - 6)
                                  for c, j in zip(codes, keys))
                        assert abs(O[b * L + i, h * dh + d] - ref) < 1e-12


def test_gelu_and_bf16_rounding_match_library():
    x = np.linspace(-6, 6, 2001)
    ref = torch.nn.functional.gelu(torch.from_numpy(x)).numpy()
    assert np.abs(orc.gelu(x) - ref).max() < 1e-15
    assert orc.gelu(np.array([0.0]))[0] == 0.0 and abs(orc.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15
    rng = np.random.default_rng(8)
    v = (rng.normal(size=20000) * 10.0 ** rng.uniform(-3, 3, 20000)).astype(np.float32)
    ref = torch.from_numpy(v).to(torch.bfloat16).float().numpy().astype(np.float64)
    assert np.array_equal(orc.round_bf16(v.astype(np.float64)), ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert orc.round_bf16(np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8])).tolist() == [1.0, 1.0 + 2 ** -6]


# ------------------------------------------------------------------ block composition (sanity, not a pin)

def test_block_error_shrinks_with_bits():
    """The quantized block approaches the full-precision block as bits grow (composition sanity)."""
    from workloads.block import _fp_forward
    errs = []
    for bits in (4, 6, 8):
        w = make_block_inputs("c1_vit_s", bits_a=bits, bits_w=bits, bits_p=bits)
        y = orc.block_forward(w)["y"]
        tp = lambda a: torch.from_numpy(a).double()
        p = {k: tp(getattr(w, k)) for k in ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_proj", "b_proj",
                                             "ln2_gamma", "ln2_beta", "w_fc1", "b_fc1", "w_fc2", "b_fc2")}
        a = _fp_forward(tp(w.x)[None], p, w.cfg)
        ref = (torch.nn.functional.linear(a["hidden"], p["w_fc2"], p["b_fc2"])[0]
               + torch.nn.functional.linear(a["attn"], p["w_proj"], p["b_proj"])[0] + tp(w.x)).numpy()
        errs.append(np.linalg.norm(y - ref) / np.linalg.norm(ref))
    assert errs[0] > errs[1] > errs[2]
    assert errs[2] < 0.05


# ------------------------------------------------------------------ block composition (pin)

def _loop_block(w):
    """Eqs. 1-3 and the quantizer placement of Sec. III-A / IV-A written out a second time, token by token, head
    by head and channel by channel, for tiny blocks.  It shares only the leaf quantizers (pinned above) with
    `block_forward`: the normalisation, the reparameterization (Eqs. 10-14), the shifted linear layer (Eq. 13,
    right-hand side), the Softmax, the rotary embedding, the non-linearities and every index are restated here
    with Python scalars."""
    import cmath
    cfg = w.cfg
    B, L, D, H, MLP = cfg["B"], cfg["L"], cfg["D"], cfg["H"], cfg["MLP"]
    ba, bw, bp = cfg["bits_a"], cfg["bits_w"], cfg["bits_p"]
    dh = D // H
    M = B * L
    llama = cfg.get("arch", "vit") == "llama"
    kept = {}

    def normalise(row, gamma, beta):
        row = [float(v) for v in row]
        mu = 0.0 if llama else sum(row) / D
        var = sum((v - mu) ** 2 for v in row) / D
        return [(v - mu) / math.sqrt(var + cfg["eps"]) * float(gamma[c]) + float(beta[c]) for c, v in enumerate(row)]

    def rtn_rows(Wm):
        q, s_w, z_w = orc.quant_weight_rtn(Wm, bw)
        return [[float(s_w[j]) * (int(q[j, c]) - int(z_w[j])) for c in range(Wm.shape[1])] for j in range(Wm.shape[0])]

    def after_norm(X_in, gamma, beta, lo, hi, W, b, tag):
        N = W.shape[0]
        s, z = orc.uniform_scale_zero(lo, hi, ba)
        s_t = sum(float(v) for v in s) / D
        z_mean = sum(int(v) for v in z) / D
        z_t = int(np.rint(z_mean))
        r1 = [float(s[c]) / s_t for c in range(D)]
        r2 = [int(z[c]) - z_t for c in range(D)]
        # W~ (stored in float32) and its channel-wise RTN de-quantization; b~ from the full-precision W
        W_t = np.array([[np.float32(r1[c] * float(W[j, c])) for c in range(D)] for j in range(N)], dtype=np.float64)
        W_hat = rtn_rows(W_t)
        b_t = [float(b[j]) - sum(float(s[c]) * r2[c] * float(W[j, c]) for c in range(D)) for j in range(N)]
        codes = np.zeros((M, D), dtype=np.int64)
        Y = np.zeros((M, N))
        for n in range(M):
            x1 = normalise(X_in[n], gamma, beta)
            for c in range(D):
                codes[n, c] = int(orc.quant_uniform(x1[c], float(s[c]), int(z[c]), ba)[0])
            x_hat = [float(s[c]) * (int(codes[n, c]) - int(z[c])) for c in range(D)]
            shifted = [(x_hat[c] + float(s[c]) * r2[c]) / r1[c] for c in range(D)]
            for j in range(N):
                Y[n, j] = sum(shifted[c] * W_hat[j][c] for c in range(D)) + b_t[j]
        kept[tag + "_codes"] = codes
        return Y

    def layerwise(V, name):
        lo, hi = w.bounds[name]
        s, z = orc.uniform_scale_zero(lo, hi, ba)
        q = np.zeros(V.shape, dtype=np.int64)
        for i in range(V.shape[0]):
            for j in range(V.shape[1]):
                q[i, j] = int(orc.quant_uniform(float(V[i, j]), float(s), int(z), ba)[0])
        kept[name + "_codes"] = q
        return q, float(s) * (q.astype(np.float64) - int(z))

    def plain_linear(X_hat, W, b):
        W_hat = rtn_rows(np.asarray(W, dtype=np.float64))
        N = W.shape[0]
        out = np.zeros((X_hat.shape[0], N))
        for n in range(X_hat.shape[0]):
            for j in range(N):
                out[n, j] = sum(float(X_hat[n, c]) * W_hat[j][c] for c in range(X_hat.shape[1])) + float(b[j])
        return out

    x = np.asarray(w.x, dtype=np.float64)
    qkv = after_norm(x, w.ln1_gamma, w.ln1_beta, w.ln1_lo, w.ln1_hi, w.w_qkv, w.b_qkv, "ln1")
    Q, K, V = qkv[:, :D].copy(), qkv[:, D:2 * D].copy(), qkv[:, 2 * D:].copy()
    if llama:
        base = cfg.get("rope_base", 10000.0)
        for T in (Q, K):
            for n in range(M):
                pos = n % L
                for h in range(H):
                    for i in range(dh // 2):
                        c0 = h * dh + 2 * i
                        zc = complex(T[n, c0], T[n, c0 + 1]) * cmath.exp(1j * pos * base ** (-2.0 * i / dh))
                        T[n, c0], T[n, c0 + 1] = zc.real, zc.imag
    _, Qh = layerwise(Q, "q")
    _, Kh = layerwise(K, "k")
    _, Vh = layerwise(V, "v")
    O = np.zeros((M, D))
    p_codes = []
    for b_ in range(B):
        for h in range(H):
            pc = np.zeros((L, L), dtype=np.int64)
            for i in range(L):
                n_keys = i + 1 if cfg["causal"] else L
                sc = [sum(Qh[b_ * L + i, h * dh + d] * Kh[b_ * L + j, h * dh + d] for d in range(dh)) / math.sqrt(dh)
                      for j in range(n_keys)]
                mx = max(sc)
                e = [math.exp(v - mx) for v in sc]
                tot = sum(e)
                for j in range(n_keys):
                    code = int(orc.quant_logsqrt2(e[j] / tot, w.softmax_scale, bp)[0])
                    pc[i, j] = code
                    a_hat = float(orc.dequant_logsqrt2(code, w.softmax_scale))
                    for d in range(dh):
                        O[b_ * L + i, h * dh + d] += a_hat * Vh[b_ * L + j, h * dh + d]
            p_codes.append(pc)
    kept["p_codes"] = p_codes
    _, Oh = layerwise(O, "attn")
    x_bar = plain_linear(Oh, w.w_proj, w.b_proj) + x
    if cfg["act"] == "bf16":
        x_bar = orc.round_bf16(x_bar)
    kept["x_bar"] = x_bar
    pre = after_norm(x_bar, w.ln2_gamma, w.ln2_beta, w.ln2_lo, w.ln2_hi, w.w_fc1, w.b_fc1, "ln2")
    if llama:
        act = np.array([[pre[n, j] / (1.0 + math.exp(-pre[n, j])) * pre[n, MLP + j] for j in range(MLP)] for n in range(M)])
    else:
        act = np.array([[0.5 * pre[n, j] * (1.0 + math.erf(pre[n, j] / math.sqrt(2.0))) for j in range(MLP)] for n in range(M)])
    _, Hh = layerwise(act, "hidden")
    kept["y"] = plain_linear(Hh, w.w_fc2, w.b_fc2) + x_bar
    return kept


def _soft_attention(w, k=7e-4):
    """The generator's attention temperature gives nearly one-hot Softmax rows at 5 tokens; scale the query
    projection (and its clipping bounds) down so that the tiny block's Softmax codes take many values."""
    import dataclasses
    D = w.cfg["D"]
    w_qkv, b_qkv = w.w_qkv.copy(), w.b_qkv.copy()
    w_qkv[:D] *= np.float32(k)
    b_qkv[:D] *= np.float32(k)
    bounds = dict(w.bounds)
    bounds["q"] = (np.float32(w.bounds["q"][0] * k), np.float32(w.bounds["q"][1] * k))
    return dataclasses.replace(w, w_qkv=w_qkv, b_qkv=b_qkv, bounds=bounds)


@pytest.mark.parametrize("name,causal,act", [
    ("c1_vit_s", False, "f32"), ("c1_vit_s", True, "bf16"), ("c4_llama7b_arch", True, "bf16"),
    ("c4_llama7b_arch", False, "f32"),
])
def test_block_forward_against_loop_written_block(name, causal, act):
    """`block_forward` against the loop-written block: the output, the residual stream and every code tensor."""
    w = _soft_attention(make_block_inputs(name, batch=2, D=8, H=2, MLP=16, L=5, causal=causal, act=act, bits_p=4,
                                          massive=1, calib_samples=32))
    got = orc.block_forward(w, keep=True)
    ref = _loop_block(w)
    L, causal_ = w.cfg["L"], w.cfg["causal"]
    checked = 0
    for key in ("ln1_codes", "q_codes", "k_codes", "v_codes", "attn_codes", "ln2_codes", "hidden_codes"):
        a, b = np.asarray(got[key]), np.asarray(ref[key])
        assert a.shape == b.shape
        if not np.array_equal(a, b):
            # the two statements round the same real number computed in two orders: a code may differ only where
            # the value handed to the round operation is a tie up to float64 round-off
            t = np.asarray(got[key[:-6] + "_t"])
            bad = (a != b) & ~((np.abs(a - b) == 1) & (np.abs(t - np.floor(t) - 0.5) < 1e-9))
            assert not bad.any(), key
        checked += a.size
    for pair, (pa, pb) in enumerate(zip(got["p_codes"], ref["p_codes"])):
        mask = np.tril(np.ones((L, L), dtype=bool)) if causal_ else np.ones((L, L), dtype=bool)
        assert np.array_equal(np.asarray(pa)[mask], pb[mask]), pair
        checked += int(mask.sum())
    assert checked > 500
    assert np.abs(got["x_bar"] - ref["x_bar"]).max() <= 1e-11 * np.abs(ref["x_bar"]).max()
    assert np.abs(got["y"] - ref["y"]).max() <= 1e-11 * np.abs(ref["y"]).max()
    # the codes are not degenerate: several distinct values per tensor, Softmax codes included
    assert len(np.unique(got["ln1_codes"])) > 4 and len(np.unique(got["hidden_codes"])) > 2
    assert len(np.unique(np.concatenate([np.asarray(p).ravel() for p in got["p_codes"]]))) > 3


def _mutated(fn_name, replacement):
    class _Swap:
        def __enter__(self):
            self.old = getattr(orc, fn_name)
            setattr(orc, fn_name, replacement)
        def __exit__(self, *a):
            setattr(orc, fn_name, self.old)
    return _Swap()


def test_loop_written_block_catches_planted_mistakes():
    """Mistakes planted in the oracle's composition (on the CPU) make the comparison above fail: a dropped bias
    compensation (Eq. 14), a missing bf16 rounding of the residual stream, swapped K / V bounds, GELU after the
    hidden quantizer instead of before it."""
    w = _soft_attention(make_block_inputs("c1_vit_s", batch=1, D=8, H=2, MLP=16, L=5, act="bf16", calib_samples=32))
    ref = _loop_block(w)
    base = orc.block_forward(w)["y"]
    assert np.abs(base - ref["y"]).max() <= 1e-11 * np.abs(ref["y"]).max()

    def differs(y):
        return np.abs(y - ref["y"]).max() > 1e-6 * np.abs(ref["y"]).max()

    real_reparam = orc.reparam_layernorm
    def no_bias_compensation(gamma, beta, s, z, W, b):
        rp = dict(real_reparam(gamma, beta, s, z, W, b))
        rp["b_t"] = np.zeros(W.shape[0]) if b is None else np.asarray(b, dtype=np.float64)
        return rp
    with _mutated("reparam_layernorm", no_bias_compensation):
        assert differs(orc.block_forward(w)["y"])
    with _mutated("round_bf16", lambda v: np.asarray(v, dtype=np.float64)):
        assert differs(orc.block_forward(w)["y"])
    import dataclasses
    swapped = dict(w.bounds)
    swapped["k"], swapped["v"] = w.bounds["v"], w.bounds["k"]
    assert differs(orc.block_forward(dataclasses.replace(w, bounds=swapped))["y"])
    real_gelu = orc.gelu
    with _mutated("gelu", lambda v: np.asarray(v, dtype=np.float64)):
        y_no_gelu = orc.block_forward(w)["y"]
    assert differs(y_no_gelu)


# ------------------------------------------------------------------ rotary embedding and SiLU (LLaMA block form)

def test_rope_against_complex_rotation_and_its_invariants():
    import cmath
    rng = np.random.default_rng(21)
    B, L, H, dh = 2, 7, 3, 8
    X = rng.normal(size=(B * L, H * dh))
    Y = orc.rope(X, B, L, H, base=10000.0)
    for n in range(B * L):
        m = n % L
        for h in range(H):
            for i in range(dh // 2):
                c0 = h * dh + 2 * i
                zc = complex(X[n, c0], X[n, c0 + 1]) * cmath.exp(1j * m * 10000.0 ** (-2.0 * i / dh))
                assert abs(Y[n, c0] - zc.real) < 1e-13 and abs(Y[n, c0 + 1] - zc.imag) < 1e-13
    # position 0 is the identity; a rotation keeps every pair's length
    assert np.array_equal(Y[0], X[0]) and np.array_equal(Y[L], X[L])
    assert np.allclose((Y.reshape(-1, 2) ** 2).sum(1), (X.reshape(-1, 2) ** 2).sum(1), rtol=1e-13)
    # relative-position property: <rope(q)_m, rope(k)_n> depends on m - n only
    q, k = rng.normal(size=(1, dh)), rng.normal(size=(1, dh))
    Qr = orc.rope(np.repeat(q, L, axis=0), 1, L, 1)
    Kr = orc.rope(np.repeat(k, L, axis=0), 1, L, 1)
    G = Qr @ Kr.T
    for d in range(-(L - 1), L):
        diag = np.diagonal(G, offset=-d)
        assert np.allclose(diag, diag[0], atol=1e-12)
    # the first pair rotates by one radian per position (theta_0 = 1)
    e0 = np.zeros((L, dh)); e0[:, 0] = 1.0
    R = orc.rope(e0, 1, L, 1)
    assert np.allclose(R[:, 0], np.cos(np.arange(L))) and np.allclose(R[:, 1], np.sin(np.arange(L)))


def test_silu_matches_library():
    x = np.linspace(-12, 12, 2401)
    ref = torch.nn.functional.silu(torch.from_numpy(x)).numpy()
    assert np.abs(orc.silu(x) - ref).max() < 1e-15
    assert orc.silu(np.array([0.0]))[0] == 0.0


def test_llama_form_reduces_to_paper_form_pieces():
    """RMS normalisation of a zero-mean row equals LayerNorm of it; rotary embedding with every token at
    position 0 (L = 1) leaves the block's attention unchanged."""
    rng = np.random.default_rng(5)
    X = rng.normal(size=(6, 16))
    X -= X.mean(axis=1, keepdims=True)
    g, b = rng.normal(size=16), rng.normal(size=16)
    assert np.allclose(orc.layernorm(X, g, b, 1e-6, rms=True), orc.layernorm(X, g, b, 1e-6), rtol=1e-12, atol=1e-12)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(X + 0.3), (16,), weight=torch.from_numpy(g), eps=1e-6).numpy() + b
    assert np.allclose(orc.layernorm(X + 0.3, g, b, 1e-6, rms=True), ref, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ per-channel dual clipping (Eqs. 18-20)

def _torch_dual_clip_loss(Xt, a1, a2, bits):
    """Eq. 20 through torch autograd: quantizer of Eqs. 4-6 on the bounds of Eqs. 18-19, round passed straight
    through (library routines: sigmoid, round, clamp, autograd)."""
    Q = 2 ** bits - 1
    up = Xt.max(0).values * torch.sigmoid(a1)
    low = Xt.min(0).values * torch.sigmoid(a2)
    s = (up - low) / Q
    ste = lambda v: (torch.round(v) - v).detach() + v
    z = ste(-low / s)
    q = torch.clamp(ste(Xt / s) + z, 0, Q)
    return ((s * (q - z) - Xt) ** 2).sum(0)


def _clip_case(seed=0, n=600, D=7):
    rng = np.random.default_rng(seed)
    X = rng.normal(size=(n, D)) * np.exp(rng.normal(0, 1, D)) + rng.normal(0, 1, D)
    X[::40, 2] *= 5.0            # one-sided outliers in one channel, two-sided in another
    X[7::55, 4] -= 6.0
    X[3::70, 4] += 9.0
    return X


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_dual_clip_loss_and_gradient_match_autograd(bits):
    X = _clip_case()
    D = X.shape[1]
    rng = np.random.default_rng(bits)
    a1n, a2n = rng.normal(0, 1.5, D), rng.normal(0, 1.5, D)
    a1 = torch.tensor(a1n, requires_grad=True)
    a2 = torch.tensor(a2n, requires_grad=True)
    L = _torch_dual_clip_loss(torch.from_numpy(X), a1, a2, bits)
    L.sum().backward()
    loss, g1, g2 = orc.dual_clip_loss_grad(X, a1n, a2n, bits)
    assert np.allclose(loss, L.detach().numpy(), rtol=1e-12)
    assert np.allclose(g1, a1.grad.numpy(), rtol=1e-9, atol=1e-9 * np.abs(g1).max())
    assert np.allclose(g2, a2.grad.numpy(), rtol=1e-9, atol=1e-9 * np.abs(g2).max())
    # the loss is the quantization error of the channel-wise quantizer built on the same bounds
    up, low = orc.dual_clip_bounds(X.max(0), X.min(0), a1n, a2n)
    s = (up - low) / (2 ** bits - 1)
    z = np.rint(-low / s)
    q, _ = orc.quant_uniform(X, s[None, :], z[None, :], bits)
    assert np.allclose(loss, ((orc.dequant_uniform(q, s[None, :], z[None, :]) - X) ** 2).sum(0), rtol=1e-12)


def test_dual_clip_follows_the_library_optimizer_and_lowers_the_objective():
    X = _clip_case(seed=1)
    D = X.shape[1]
    a1 = torch.zeros(D, dtype=torch.float64, requires_grad=True)
    a2 = torch.zeros(D, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([a1, a2], lr=0.01)
    Xt = torch.from_numpy(X)
    for _ in range(100):
        opt.zero_grad()
        _torch_dual_clip_loss(Xt, a1, a2, 4).sum().backward()
        opt.step()
    r = orc.dual_clip(X, 4, iters=100, lr=0.01, alpha0=0.0)
    assert np.abs(r["alpha1"] - a1.detach().numpy()).max() < 1e-9
    assert np.abs(r["alpha2"] - a2.detach().numpy()).max() < 1e-9
    assert np.all(r["loss"] < r["loss0"])
    up, low = orc.dual_clip_bounds(X.max(0), X.min(0), r["alpha1"], r["alpha2"])
    assert np.array_equal(up, r["x_up"]) and np.array_equal(low, r["x_low"])
    assert np.all(r["x_up"] <= X.max(0)) and np.all(r["x_low"] >= X.min(0))        # a contraction of the extremes
    # zero iterations: the initial contraction itself
    r0 = orc.dual_clip(X, 4, iters=0, alpha0=0.0)
    assert np.allclose(r0["x_up"], 0.5 * X.max(0)) and np.allclose(r0["x_low"], 0.5 * X.min(0))


def test_dual_clip_beats_the_percentile_stand_in_on_layernorm_activations():
    """On the LayerNorm activations of a seeded calibration batch, the learned per-channel bounds give a smaller
    objective (Eq. 20) than the 0.1 / 99.9 percentile bounds the workloads use in their place."""
    from workloads.kernels import affine_params, channel_profile, ln_inputs, percentile_bounds
    rng = np.random.default_rng(11)
    D = 48
    c, shift = channel_profile(rng, D, 1.0, 0.04, 20.0)
    gamma, beta = affine_params(rng, D)
    X1 = orc.layernorm(ln_inputs(rng, 1500, c, shift, False), gamma, beta, 1e-6)
    lo, hi = percentile_bounds(X1, axis=0)
    s, z = orc.uniform_scale_zero(lo, hi, 4)
    q, _ = orc.quant_uniform(X1, s[None, :], z[None, :], 4)
    err_pct = ((orc.dequant_uniform(q, s[None, :], z[None, :]) - X1) ** 2).sum()
    r = orc.dual_clip(X1, 4, alpha0=2.0)            # start at 0.88 of the extremes
    assert r["loss"].sum() < err_pct
    assert r["loss"].sum() < r["loss0"].sum()
