"""Shared helpers of the GPU parity tests and of the smoke check: code unpacking, the near-tie
protocol, float tolerances, and stage-level comparisons between the CUDA path and the CPU oracle."""
from __future__ import annotations

import math

import numpy as np

REL_L2_TOL = 2e-3          # float outputs: relative L2 error
MAX_ABS_TOL = 1e-2         # float outputs: max abs error as a fraction of max |ref|


BYTE_CODES = 0x100         # flag of the C ABI: a `bits` value with it set stores one code per byte


def qb(bits: int) -> int:
    """Quantizer width of a `bits` value (the flag only changes the storage)."""
    return bits & 0xFF


def unpack_codes(raw: np.ndarray, n: int, bits: int) -> np.ndarray:
    """raw: uint8 [rows, ld_bytes] -> int64 [rows, n] (4-bit: low nibble = even index)."""
    raw = np.asarray(raw, dtype=np.uint8)
    if bits == 4:
        lo = raw & 0x0F
        hi = raw >> 4
        out = np.stack([lo, hi], axis=-1).reshape(raw.shape[0], -1)
    else:
        out = raw
    return out[:, :n].astype(np.int64)


def pack_codes(q: np.ndarray, bits: int, ld_bytes: int) -> np.ndarray:
    """int codes [rows, n] -> uint8 [rows, ld_bytes] in the library's layout (test-side packing)."""
    q = np.asarray(q, dtype=np.uint8)
    rows, n = q.shape
    out = np.zeros((rows, ld_bytes), dtype=np.uint8)
    if bits == 4:
        if n % 2:
            q = np.concatenate([q, np.zeros((rows, 1), dtype=np.uint8)], axis=1)
        out[:, : q.shape[1] // 2] = q[:, 0::2] | (q[:, 1::2] << 4)
    else:
        out[:, :n] = q
    return out


def near_tie_report(q_gpu: np.ndarray, q_ref: np.ndarray, t_ref: np.ndarray, delta) -> dict:
    """Bit-exactness of integer codes decided in float32 on the GPU and float64 in the oracle.

    A mismatch is excused only if it is +-1 and the oracle's pre-rounding value t lies within `delta`
    of a rounding tie (x.5).  Returns counts; `bad` must be 0.
    """
    q_gpu = np.asarray(q_gpu, dtype=np.int64)
    q_ref = np.asarray(q_ref, dtype=np.int64)
    diff = q_gpu != q_ref
    n_mis = int(diff.sum())
    if n_mis == 0:
        return dict(total=q_ref.size, mismatch=0, excused=0, bad=0)
    t = np.asarray(t_ref, dtype=np.float64)[diff]
    d = np.broadcast_to(np.asarray(delta, dtype=np.float64), q_ref.shape)[diff]
    with np.errstate(invalid="ignore"):
        dist = np.abs(t - np.floor(t) - 0.5)
    ok = (np.abs(q_gpu[diff] - q_ref[diff]) == 1) & (dist < d)
    return dict(total=q_ref.size, mismatch=n_mis, excused=int(ok.sum()), bad=int((~ok).sum()))


def float_errors(out: np.ndarray, ref: np.ndarray):
    out = np.asarray(out, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rel_l2 = float(np.linalg.norm(out - ref) / max(np.linalg.norm(ref), 1e-300))
    max_abs = float(np.abs(out - ref).max() / max(np.abs(ref).max(), 1e-300))
    return rel_l2, max_abs


def assert_float_close(out, ref, what=""):
    rel_l2, max_abs = float_errors(out, ref)
    assert rel_l2 <= REL_L2_TOL and max_abs <= MAX_ABS_TOL, "%s rel_l2=%.3e max_abs/max|ref|=%.3e" % (what, rel_l2, max_abs)
    return rel_l2, max_abs


# ------------------------------------------------------------------------------------------ stages

def ln_case(rows: int, D: int, bf16: bool, seed: int, rms: bool = False, eps: float = 1e-6):
    from workloads.kernels import affine_params, channel_profile, ln_calibration_bounds, ln_inputs
    rng = np.random.default_rng(seed)
    c, shift = channel_profile(rng, D, 1.0, 0.01, 50.0)
    gamma, beta = affine_params(rng, D)
    x_cal = ln_inputs(rng, 2048, c, shift, bf16)
    x = ln_inputs(rng, rows, c, shift, bf16)
    lo, hi = ln_calibration_bounds(x_cal, gamma, beta, eps, rms)
    return x, gamma, beta, lo, hi


def ln_delta(x, gamma_t, s_t, t_lw, eps, rms):
    """Near-tie width for the fused LN+quant kernel: float32 rounding of (x - mu) * rstd * gamma~/s~ + beta~/s~.
    The subtraction carries about 2^-22 |mu| (rounded mean) and the products 2^-23 relative each; the bound
    below leaves a factor of 8 over that."""
    x = np.asarray(x, dtype=np.float64)
    mu = np.zeros((x.shape[0], 1)) if rms else x.mean(axis=1, keepdims=True)
    d = x - mu
    rstd = 1.0 / np.sqrt((d * d).mean(axis=1, keepdims=True) + eps)
    return 2.0 ** -19 * (np.abs(x) + np.abs(mu)) * rstd * np.abs(gamma_t)[None, :] / s_t + 2.0 ** -20 * np.abs(t_lw)


def check_ln_quant(rows, D, bits, bf16, seed=0, rms=False, eps=1e-6, pad_cols=0, want_sum=True):
    """Runs the fused LN+quant kernel and compares its codes with the oracle's channel-wise codes."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    x, gamma, beta, lo, hi = ln_case(rows, D, bf16, seed, rms, eps)
    # oracle: complex (channel-wise) quantizer
    X1 = orc.layernorm(x, gamma, beta, eps, rms)
    s, z = orc.uniform_scale_zero(lo, hi, qb(bits))
    q_ref, t_cw = orc.quant_uniform(X1, s[None, :], z[None, :], qb(bits))
    # CUDA path: folded parameters, layer-wise quantizer
    W = np.zeros((1, D), dtype=np.float32)
    gamma_t, beta_t, s_t, z_t, _, _ = B.repq_fold_ln(gamma, beta, s.astype(np.float32), z.astype(np.int32), W, None)
    dev = torch.device("cuda:0")
    xt = torch.from_numpy(x).to(dev)
    if bf16:
        xt = xt.to(torch.bfloat16)
    if pad_cols:
        buf = torch.zeros(rows, D + pad_cols, dtype=xt.dtype, device=dev)
        buf[:, :D] = xt
        xt = buf[:, :D]
    ld = B.code_row_bytes(D, bits)
    codes = torch.full((max(rows, 1), ld), 0xEE, dtype=torch.uint8, device=dev)[:rows]
    row_sum = torch.full((max(rows, 1),), -1, dtype=torch.int32, device=dev)[:rows] if want_sum else None
    B.repq_ln_quant(xt, torch.from_numpy(gamma_t).to(dev), torch.from_numpy(beta_t).to(dev), eps, s_t, z_t, bits,
                    codes, row_sum, B.REPQ_NORM_RMS if rms else B.REPQ_NORM_LAYERNORM)
    torch.cuda.synchronize()
    if rows == 0:
        return dict(total=0, mismatch=0, excused=0, bad=0)
    q_gpu = unpack_codes(codes.cpu().numpy(), D, bits)
    t_lw = t_cw + (z - z_t)[None, :]
    rep = near_tie_report(q_gpu, q_ref, t_cw, ln_delta(x, gamma_t.astype(np.float64), s_t, t_lw, eps, rms))
    if want_sum:
        assert np.array_equal(row_sum.cpu().numpy().astype(np.int64), q_gpu.sum(axis=1)), "row sums"
    # bytes beyond the row's codes are untouched
    raw = codes.cpu().numpy()
    used = D // 2 if bits == 4 else D
    assert np.all(raw[:, used:] == 0xEE)
    return rep


def check_softmax_log2(rows, L, bits, bf16=False, seed=0, s=1.0, causal_period=0, pre_scale=1.0, ld_pad=None):
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import softmax_logits, to_bf16_grid

    rng = np.random.default_rng(seed)
    S = softmax_logits(rng, rows, L)
    if bf16:
        S = to_bf16_grid(S)
    valid = None
    if causal_period:
        valid = np.minimum(L, (np.arange(rows) % causal_period) + 1)
    A = orc.softmax_rows(S.astype(np.float64) * np.float64(np.float32(pre_scale)), valid)
    q_ref, t_ref = orc.quant_logsqrt2(A, s, qb(bits))
    dev = torch.device("cuda:0")
    ld = ld_pad if ld_pad is not None else (L + 3) // 4 * 4
    buf = torch.zeros(rows, ld, dtype=torch.float32, device=dev)
    buf[:, :L] = torch.from_numpy(S).to(dev)
    if bf16:
        buf = buf.to(torch.bfloat16)
    unit = 4 if bits == 4 else 8
    ldc = max(B.code_row_bytes(L, bits), (L + 7) // 8 * unit)
    codes = torch.full((rows, ldc), 0xEE, dtype=torch.uint8, device=dev)
    B.repq_softmax_log2(buf, L, s, bits, codes, pre_scale, causal_period, 0)
    torch.cuda.synchronize()
    q_gpu = unpack_codes(codes.cpu().numpy(), L, bits)
    delta = 2.0 ** -18 * np.maximum(1.0, np.abs(np.where(np.isfinite(t_ref), t_ref, 0.0)))
    if valid is not None:
        mask = np.arange(L)[None, :] < valid[:, None]
        assert np.all(q_gpu[~mask] == 2 ** qb(bits) - 1)
        q_gpu = np.where(mask, q_gpu, 0)
        q_ref = np.where(mask, q_ref, 0)
    return near_tie_report(q_gpu, q_ref, t_ref, delta)


def smoke_check():
    rep = check_ln_quant(rows=197, D=384, bits=4, bf16=False, seed=0)
    assert rep["bad"] == 0, rep
    rep = check_softmax_log2(rows=197 * 6, L=197, bits=4, seed=0)
    assert rep["bad"] == 0, rep
    check_block("c1_vit_s", batch=1)


def check_qgemm(M, N, K, bits_a, bits_w, out_kind="f32", gelu=False, residual=None, groups=1, out_bits=4, seed=0,
                want_acc=True, want_out_sum=False, give_sums=False):
    """repq_qgemm against the oracle: int32 accumulators bit-exact vs the int64 brute force, float outputs within
    tolerance, re-quantized codes bit-exact up to counted near-ties."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import gemm_codes, to_bf16_grid

    rng = np.random.default_rng(seed)
    a, w, s_a, z_a, s_w, z_w, bias = gemm_codes(rng, M, N, K, qb(bits_a), qb(bits_w))
    res = None
    if residual is not None:
        res = rng.normal(0, 1.0, size=(M, N)).astype(np.float32)
        if residual == "bf16":
            res = to_bf16_grid(res)
    # ---- oracle
    acc_ref = orc.int_gemm(a, w)
    v_pre = orc.linear(orc.dequant_uniform(a, s_a, z_a), w, s_w, z_w, bias)
    v_ref = orc.gelu(v_pre) if gelu else v_pre
    if res is not None:
        v_ref = v_ref + res
    # ---- CUDA path
    dev = torch.device("cuda:0")
    lda, ldw = B.code_row_bytes(K, bits_a), B.code_row_bytes(K, bits_w)
    a_t = torch.from_numpy(pack_codes(a, bits_a, lda)).to(dev)
    w_t = torch.from_numpy(pack_codes(w, bits_w, ldw)).to(dev)
    kw = {}
    if out_kind == "codes":
        gw = N // groups
        lo = [np.percentile(v_ref[:, g * gw:(g + 1) * gw], 1) for g in range(groups)]
        hi = [np.percentile(v_ref[:, g * gw:(g + 1) * gw], 99) for g in range(groups)]
        s_o, z_o = orc.uniform_scale_zero(np.array(lo), np.array(hi), qb(out_bits))
        ldo = B.code_row_bytes(N, out_bits)
        out = torch.full((M, ldo), 0xEE, dtype=torch.uint8, device=dev)
        kw = dict(out_kind=B.REPQ_OUT_CODES, out_bits=out_bits, out_scale=[float(v) for v in s_o],
                  out_zero=[int(v) for v in z_o])
        if want_out_sum:
            kw["out_row_sum"] = torch.zeros(M, dtype=torch.int32, device=dev)
    elif out_kind == "bf16":
        out = torch.zeros(M, N, dtype=torch.bfloat16, device=dev)
        kw = dict(out_kind=B.REPQ_OUT_BF16)
    else:
        out = torch.zeros(M, N, dtype=torch.float32, device=dev)
    acc = torch.zeros(M, N, dtype=torch.int32, device=dev) if want_acc else None
    res_t = None
    if res is not None:
        res_t = torch.from_numpy(res).to(dev)
        if residual == "bf16":
            res_t = res_t.to(torch.bfloat16)
    if give_sums:
        kw["a_row_sum"] = torch.from_numpy(a.sum(axis=1).astype(np.int32)).to(dev)
        kw["w_row_sum"] = torch.from_numpy(w.sum(axis=1).astype(np.int32)).to(dev)
    # the descriptor holds raw pointers: keep every tensor alive until the call has run
    s_w_t, z_w_t, bias_t = (torch.from_numpy(v).to(dev) for v in (s_w, z_w, bias))
    d = B.gemm_desc(M, N, K, a_t, bits_a, float(s_a), int(z_a), w_t, bits_w, out,
                    s_w=s_w_t, z_w=z_w_t, bias=bias_t, gelu=gelu, residual=res_t, acc_debug=acc, **kw)
    nws = B.repq_qgemm_workspace_bytes(d)
    ws = torch.empty(max(nws, 16), dtype=torch.uint8, device=dev)
    B.repq_qgemm(d, ws)
    torch.cuda.synchronize()
    assert B.repq_device_status() == 0
    result = {}
    if want_acc:
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref), "int32 accumulators differ from brute force"
    if out_kind == "codes":
        gw = N // groups
        q_gpu = unpack_codes(out.cpu().numpy(), N, out_bits)
        rep = dict(total=0, mismatch=0, excused=0, bad=0)
        for g in range(groups):
            sl = slice(g * gw, (g + 1) * gw)
            q_ref, t_ref = orc.quant_uniform(v_ref[:, sl], s_o[g], z_o[g], qb(out_bits))
            mag = np.abs(v_pre[:, sl] - bias[None, sl]) + np.abs(bias[None, sl]) + np.abs(v_ref[:, sl])
            if res is not None:
                mag = mag + np.abs(res[:, sl])
            delta = 2.0 ** -19 * mag / s_o[g] + 2.0 ** -20 * np.abs(t_ref)
            r = near_tie_report(q_gpu[:, sl], q_ref, t_ref, delta)
            for k in rep:
                rep[k] += r[k]
        assert rep["bad"] == 0, rep
        if want_out_sum:
            assert np.array_equal(kw["out_row_sum"].cpu().numpy().astype(np.int64), q_gpu.sum(axis=1))
        result = rep
    else:
        got = out.float().cpu().numpy()
        if out_kind == "bf16":
            # bf16 output = RNE(float32 value): compare against the oracle rounded the same way, 1 bf16 ulp
            # (a residual that cancels the GEMM value leaves the float32 rounding of the two addends, 2^-23
            # relative to each, which no rounding of the small sum can undo: allowed in absolute terms)
            ref16 = orc.round_bf16(v_ref)
            addends = np.abs(v_ref - res) + np.abs(res) if res is not None else 0.0
            assert np.all(np.abs(got - ref16) <= np.abs(ref16) * 2.0 ** -7 + addends * 2.0 ** -22 + 1e-30)
            rel, mx = float_errors(got, v_ref)
            assert rel < 4e-3
        else:
            rel, mx = assert_float_close(got, v_ref, "qgemm")
            assert rel < 1e-5, rel          # float32 epilogue on exact integers: far inside the tolerance
        result = dict(rel_l2=rel, max_abs=mx)
    return result


def check_pv(B_, H, Lq, Lk, dh, bits_p, bits_v, causal=False, out_kind="f32", out_bits=4, seed=0, s_p=1.0,
             want_out_sum=False):
    """repq_pv against the oracle: log-sqrt2 de-quantization (Eq. 16, first line) times de-quantized V."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import softmax_logits

    rng = np.random.default_rng(seed)
    pairs = B_ * H
    shift = Lk - Lq
    valid = np.minimum(Lk, np.arange(Lq) + 1 + shift) if causal else None
    S = softmax_logits(rng, pairs * Lq, Lk)
    A = orc.softmax_rows(S, None if valid is None else np.tile(valid, pairs))
    p, _ = orc.quant_logsqrt2(A, s_p, qb(bits_p))                        # [pairs*Lq, Lk]
    D = H * dh
    Vc = rng.integers(0, 1 << qb(bits_v), size=(B_ * Lk, D))
    s_v = 0.05
    z_v = int(rng.integers(0, 1 << qb(bits_v)))
    A_hat = orc.dequant_logsqrt2(p, s_p)
    if causal:
        A_hat = np.where(np.arange(Lk)[None, :] < np.tile(valid, pairs)[:, None], A_hat, 0.0)
    V_hat = orc.dequant_uniform(Vc, s_v, z_v)
    O_ref = np.empty((B_ * Lq, D))
    for b in range(B_):
        for h in range(H):
            pr = (b * H + h) * Lq
            O_ref[b * Lq:(b + 1) * Lq, h * dh:(h + 1) * dh] = A_hat[pr:pr + Lq] @ V_hat[b * Lk:(b + 1) * Lk, h * dh:(h + 1) * dh]
    dev = torch.device("cuda:0")
    ldp = B.code_row_bytes(Lk, bits_p)
    ldv = B.code_row_bytes(D, bits_v)
    p_t = torch.from_numpy(pack_codes(p, bits_p, ldp)).to(dev)
    v_t = torch.from_numpy(pack_codes(Vc, bits_v, ldv)).to(dev)
    d = B.PvDesc()
    d.batch_outer, d.batch_inner, d.Lq, d.Lk, d.d_h = B_, H, Lq, Lk, dh
    d.p_codes, d.bits_p, d.ldp_bytes, d.p_stride_pair, d.s_p = p_t.data_ptr(), bits_p, ldp, Lq * ldp, s_p
    d.v_codes, d.bits_v, d.ldv_bytes = v_t.data_ptr(), bits_v, ldv
    d.v_stride_outer, d.v_stride_inner = Lk * ldv, (dh // 2 if bits_v == 4 else dh)
    d.s_v, d.z_v, d.causal = s_v, z_v, int(causal)
    row_sum = None
    if out_kind == "codes":
        s_o, z_o = orc.uniform_scale_zero(np.percentile(O_ref, 1), np.percentile(O_ref, 99), qb(out_bits))
        ldo = B.code_row_bytes(D, out_bits)
        out = torch.full((B_ * Lq, ldo), 0xEE, dtype=torch.uint8, device=dev)
        d.out_kind, d.out_bits, d.out_scale, d.out_zero = B.REPQ_OUT_CODES, out_bits, float(s_o), int(z_o)
        d.ldo, d.o_stride_outer, d.o_stride_inner = ldo, Lq * ldo, (dh // 2 if out_bits == 4 else dh)
        if want_out_sum:
            row_sum = torch.zeros(B_ * Lq, dtype=torch.int32, device=dev)
            d.out_row_sum = row_sum.data_ptr()
    else:
        dt = torch.float32 if out_kind == "f32" else torch.bfloat16
        out = torch.zeros(B_ * Lq, D, dtype=dt, device=dev)
        d.out_kind = B.REPQ_OUT_F32 if out_kind == "f32" else B.REPQ_OUT_BF16
        d.ldo, d.o_stride_outer, d.o_stride_inner = D, Lq * D, dh
    d.out = out.data_ptr()
    B.repq_pv(d)
    torch.cuda.synchronize()
    if out_kind == "codes":
        q_gpu = unpack_codes(out.cpu().numpy(), D, out_bits)
        q_ref, t_ref = orc.quant_uniform(O_ref, s_o, z_o, qb(out_bits))
        absO = np.empty_like(O_ref)
        for b in range(B_):
            for h in range(H):
                pr = (b * H + h) * Lq
                absO[b * Lq:(b + 1) * Lq, h * dh:(h + 1) * dh] = A_hat[pr:pr + Lq] @ np.abs(V_hat[b * Lk:(b + 1) * Lk, h * dh:(h + 1) * dh])
        delta = 2.0 ** -18 * absO / s_o + 2.0 ** -20 * np.abs(t_ref)
        rep = near_tie_report(q_gpu, q_ref, t_ref, delta)
        assert rep["bad"] == 0, rep
        if want_out_sum:
            assert np.array_equal(row_sum.cpu().numpy().astype(np.int64), q_gpu.sum(axis=1))
        return rep
    got = out.float().cpu().numpy()
    if out_kind == "bf16":
        ref16 = orc.round_bf16(O_ref)
        assert np.all(np.abs(got - ref16) <= np.abs(ref16) * 2.0 ** -7 + 1e-30)
        return dict(rel_l2=float_errors(got, O_ref)[0])
    rel, mx = assert_float_close(got, O_ref, "pv")
    assert rel < 1e-5, rel
    return dict(rel_l2=rel, max_abs=mx)


def check_block(name, batch, sample_items=None, out_dtype="f32", staged_attention=False, **overrides):
    """Free-running block: the CUDA path (folded parameters, simple quantizers) against the oracle (complex
    quantizers) on the block output, for the sampled batch items (items are independent, Eqs. 1-3)."""
    import dataclasses
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200.engine import QuantBlock
    from workloads import make_block_inputs

    w = make_block_inputs(name, batch=batch, **overrides)
    L = w.cfg["L"]
    blk = QuantBlock(w, out_dtype=torch.float32 if out_dtype == "f32" else torch.bfloat16, staged_attention=staged_attention)
    x = torch.from_numpy(w.x).to(blk.device).to(blk.act_dtype)
    y = blk.forward(x)
    torch.cuda.synchronize()
    y = y.float().cpu().numpy()
    assert np.all(np.isfinite(y))
    items = list(range(batch)) if sample_items is None else list(sample_items)
    rows = np.concatenate([np.arange(i * L, (i + 1) * L) for i in items])
    cfg = dict(w.cfg)
    cfg["B"] = len(items)
    w_s = dataclasses.replace(w, cfg=cfg, x=w.x[rows])
    ref = orc.block_forward(w_s)["y"]
    got = y[rows]
    if out_dtype == "bf16":
        rel, mx = float_errors(got, ref)
        assert rel < 6e-3, rel
        return rel, mx
    return assert_float_close(got, ref, "block %s" % name)


def check_scores(B_, H, Lq, Lk, dh, bits, causal=False, seed=0):
    """Batched code-by-code product (attention scores) against the oracle: de-quantized Q times de-quantized
    K^T over the head dimension, scaled by 1/sqrt(d_h)."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    rng = np.random.default_rng(seed)
    D = H * dh
    Qc = rng.integers(0, 1 << qb(bits), size=(B_ * Lq, D))
    Kc = rng.integers(0, 1 << qb(bits), size=(B_ * Lk, D))
    s_q, s_k = 0.37, 0.21
    z_q, z_k = int(rng.integers(0, 1 << qb(bits))), int(rng.integers(0, 1 << qb(bits)))
    Qh, Kh = orc.dequant_uniform(Qc, s_q, z_q), orc.dequant_uniform(Kc, s_k, z_k)
    dev = torch.device("cuda:0")
    ld = B.code_row_bytes(D, bits)
    q_t = torch.from_numpy(pack_codes(Qc, bits, ld)).to(dev)
    k_t = torch.from_numpy(pack_codes(Kc, bits, ld)).to(dev)
    ld_s = (Lk + 3) // 4 * 4
    out = torch.full((B_ * H * Lq, ld_s), float("nan"), dtype=torch.float32, device=dev)
    hb = dh // 2 if bits == 4 else dh
    d = B.gemm_desc(Lq, Lk, dh, q_t, bits, s_q, z_q, k_t, bits, out, s_w_scalar=s_k, z_w_scalar=z_k,
                    alpha=1.0 / math.sqrt(dh), batch=(B_, H), a_strides=(Lq * ld, hb), w_strides=(Lk * ld, hb),
                    o_strides=(H * Lq * ld_s, Lq * ld_s), causal=causal)
    assert B.repq_qgemm_workspace_bytes(d) == 0
    B.repq_qgemm(d, None)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    worst = 0.0
    for b in range(B_):
        for h in range(H):
            ref = Qh[b * Lq:(b + 1) * Lq, h * dh:(h + 1) * dh] @ Kh[b * Lk:(b + 1) * Lk, h * dh:(h + 1) * dh].T / math.sqrt(dh)
            g = got[(b * H + h) * Lq:(b * H + h + 1) * Lq, :Lk]
            if causal:
                mask = np.arange(Lk)[None, :] <= (np.arange(Lq)[:, None] + Lk - Lq)
                g, ref = np.where(mask, g, 0.0), np.where(mask, ref, 0.0)
            assert np.all(np.isfinite(g))
            rel, _ = assert_float_close(g, ref, "scores")
            worst = max(worst, rel)
    assert worst < 1e-5
    return worst


def check_pv_uniform_codes(B_, H, L, dh, bits_p, bits_v, runs=10, seed=0):
    """repq_pv on uniformly random Softmax codes (every key carries weight, so a single misplaced tile row
    shows), launched `runs` times: every launch must reproduce the oracle and the first launch bit for bit."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    rng = np.random.default_rng(seed)
    D = H * dh
    p = rng.integers(0, 1 << qb(bits_p), size=(B_ * H * L, L))
    Vc = rng.integers(0, 1 << qb(bits_v), size=(B_ * L, D))
    s_p, s_v = 0.9, 0.05
    z_v = int(rng.integers(0, 1 << qb(bits_v)))
    A_hat = orc.dequant_logsqrt2(p, s_p)
    V_hat = orc.dequant_uniform(Vc, s_v, z_v)
    O_ref = np.empty((B_ * L, D))
    for b in range(B_):
        for h in range(H):
            pr = (b * H + h) * L
            O_ref[b * L:(b + 1) * L, h * dh:(h + 1) * dh] = A_hat[pr:pr + L] @ V_hat[b * L:(b + 1) * L, h * dh:(h + 1) * dh]
    dev = torch.device("cuda:0")
    ldp, ldv = B.code_row_bytes(L, bits_p), B.code_row_bytes(D, bits_v)
    p_t = torch.from_numpy(pack_codes(p, bits_p, ldp)).to(dev)
    v_t = torch.from_numpy(pack_codes(Vc, bits_v, ldv)).to(dev)
    out = torch.zeros(B_ * L, D, dtype=torch.float32, device=dev)
    d = B.PvDesc()
    d.batch_outer, d.batch_inner, d.Lq, d.Lk, d.d_h = B_, H, L, L, dh
    d.p_codes, d.bits_p, d.ldp_bytes, d.p_stride_pair, d.s_p = p_t.data_ptr(), bits_p, ldp, L * ldp, s_p
    d.v_codes, d.bits_v, d.ldv_bytes = v_t.data_ptr(), bits_v, ldv
    d.v_stride_outer, d.v_stride_inner = L * ldv, (dh // 2 if bits_v == 4 else dh)
    d.s_v, d.z_v, d.causal = s_v, z_v, 0
    d.out_kind = B.REPQ_OUT_F32
    d.ldo, d.o_stride_outer, d.o_stride_inner = D, L * D, dh
    d.out = out.data_ptr()
    first = None
    for _ in range(runs):
        out.zero_()
        B.repq_pv(d)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        rel, _ = assert_float_close(got, O_ref, "pv, uniform codes")
        assert rel < 1e-5, rel
        if first is None:
            first = got
        assert np.array_equal(got, first), "launches differ"
    assert B.repq_device_status() == 0


def check_attention(B_, H, Lq, Lk, dh, bits, bits_p, causal=False, out_kind="f32", out_bits=4 | BYTE_CODES, seed=0, s_p=1.0):
    """repq_attention (scores, Softmax, log-sqrt2 codes and P.V fused) against the oracle's chain of the same
    steps.  A Softmax code that sits on a rounding tie may legitimately differ by one (the near-tie protocol);
    such a flip changes a whole output row, so rows that hold a near-tie are counted and left out of the strict
    comparison."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    rng = np.random.default_rng(seed)
    D = H * dh
    nq = 1 << qb(bits)
    Qc = rng.integers(0, nq, size=(B_ * Lq, D))
    Kc = rng.integers(0, nq, size=(B_ * Lk, D))
    Vc = rng.integers(0, nq, size=(B_ * Lk, D))
    z_q, z_k, z_v = (int(rng.integers(0, nq)) for _ in range(3))
    sig = (nq / 3.5) ** 2 * math.sqrt(dh)                 # rough std of sum (q - z_q)(k - z_k)
    s_q = s_k = math.sqrt(3.0 * math.sqrt(dh) / sig)      # logits with a standard deviation of about 3
    s_v = 0.05
    alpha = 1.0 / math.sqrt(dh)
    Qh, Kh, Vh = orc.dequant_uniform(Qc, s_q, z_q), orc.dequant_uniform(Kc, s_k, z_k), orc.dequant_uniform(Vc, s_v, z_v)
    shift = Lk - Lq
    valid = np.minimum(Lk, np.arange(Lq) + 1 + shift) if causal else np.full(Lq, Lk)
    O_ref = np.empty((B_ * Lq, D))
    absO = np.empty_like(O_ref)
    tie_rows = np.zeros(B_ * Lq, dtype=bool)
    for b in range(B_):
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            S = Qh[b * Lq:(b + 1) * Lq, sl] @ Kh[b * Lk:(b + 1) * Lk, sl].T * alpha
            # the GPU forms S in float32 from the exact integer sum: do the same before the Softmax
            S = S.astype(np.float32).astype(np.float64)
            A = orc.softmax_rows(S, valid)
            p, t = orc.quant_logsqrt2(A, s_p, qb(bits_p))
            mask = np.arange(Lk)[None, :] < valid[:, None]
            tf = np.where(mask & np.isfinite(t), t, 0.25)
            near = mask & (np.abs(tf - np.floor(tf) - 0.5) < 2.0 ** -18 * np.maximum(1.0, np.abs(tf))) & (tf < min(2 ** qb(bits_p) - 0.4, 40.0))     # a flip below a weight of 2^-20 is invisible
            tie_rows[b * Lq:(b + 1) * Lq] |= near.any(axis=1)
            A_hat = np.where(mask, orc.dequant_logsqrt2(p, s_p), 0.0)
            O_ref[b * Lq:(b + 1) * Lq, sl] = A_hat @ Vh[b * Lk:(b + 1) * Lk, sl]
            absO[b * Lq:(b + 1) * Lq, sl] = A_hat @ np.abs(Vh[b * Lk:(b + 1) * Lk, sl])
    dev = torch.device("cuda:0")
    byte_bits = qb(bits) | BYTE_CODES
    q_t = torch.from_numpy(Qc.astype(np.uint8)).to(dev)
    k_t = torch.from_numpy(Kc.astype(np.uint8)).to(dev)
    v_t = torch.from_numpy(Vc.astype(np.uint8)).to(dev)
    d = B.AttentionDesc()
    d.batch_outer, d.batch_inner, d.Lq, d.Lk, d.d_h, d.bits_qkv = B_, H, Lq, Lk, dh, byte_bits
    d.q_codes, d.ldq_bytes, d.q_stride_outer, d.q_stride_inner, d.s_q, d.z_q = q_t.data_ptr(), D, Lq * D, dh, s_q, z_q
    d.k_codes, d.ldk_bytes, d.k_stride_outer, d.k_stride_inner, d.s_k, d.z_k = k_t.data_ptr(), D, Lk * D, dh, s_k, z_k
    d.v_codes, d.ldv_bytes, d.v_stride_outer, d.v_stride_inner, d.s_v, d.z_v = v_t.data_ptr(), D, Lk * D, dh, s_v, z_v
    d.alpha, d.causal, d.bits_p, d.s_p = alpha, int(causal), bits_p, s_p
    row_sum = None
    if out_kind == "codes":
        s_o, z_o = orc.uniform_scale_zero(np.percentile(O_ref, 1), np.percentile(O_ref, 99), qb(out_bits))
        ldo = B.code_row_bytes(D, out_bits)
        out = torch.full((B_ * Lq, ldo), 0xEE, dtype=torch.uint8, device=dev)
        d.out_kind, d.out_bits, d.out_scale, d.out_zero = B.REPQ_OUT_CODES, out_bits, float(s_o), int(z_o)
        d.ldo, d.o_stride_outer, d.o_stride_inner = ldo, Lq * ldo, (dh // 2 if out_bits == 4 else dh)
        row_sum = torch.zeros(B_ * Lq, dtype=torch.int32, device=dev)
        d.out_row_sum = row_sum.data_ptr()
    else:
        out = torch.zeros(B_ * Lq, D, dtype=torch.float32 if out_kind == "f32" else torch.bfloat16, device=dev)
        d.out_kind = B.REPQ_OUT_F32 if out_kind == "f32" else B.REPQ_OUT_BF16
        d.ldo, d.o_stride_outer, d.o_stride_inner = D, Lq * D, dh
    d.out = out.data_ptr()
    first = None
    for _ in range(3):                                   # repeated launches must agree bit for bit
        if row_sum is not None:
            row_sum.zero_()
        B.repq_attention(d)
        torch.cuda.synchronize()
        got_raw = out.cpu().numpy() if out_kind != "bf16" else out.float().cpu().numpy()
        if first is None:
            first = got_raw.copy()
        assert np.array_equal(got_raw, first), "launches differ"
    assert B.repq_device_status() == 0
    keep = ~tie_rows
    assert keep.mean() > 0.9, "too many rows with a Softmax code on a rounding tie: %.3f" % (1 - keep.mean())
    if out_kind == "codes":
        q_gpu = unpack_codes(first, D, out_bits)
        q_ref, t_ref = orc.quant_uniform(O_ref, s_o, z_o, qb(out_bits))
        delta = 2.0 ** -17 * absO / s_o + 2.0 ** -20 * np.abs(t_ref)
        rep = near_tie_report(q_gpu[keep], q_ref[keep], t_ref[keep], delta[keep])
        assert rep["bad"] == 0, rep
        assert np.array_equal(row_sum.cpu().numpy().astype(np.int64), q_gpu.sum(axis=1))
        return rep
    got = first.astype(np.float64)
    if out_kind == "bf16":
        rel, _ = float_errors(got[keep], O_ref[keep])
        assert rel < 6e-3, rel
        return dict(rel_l2=rel)
    rel, mx = assert_float_close(got[keep], O_ref[keep], "attention")
    assert rel < 1e-4, rel                               # exact operands, float32 sums: far inside the tolerance
    return dict(rel_l2=rel, max_abs=mx, tie_rows=int(tie_rows.sum()))
