"""Shared helpers of the GPU parity tests and of the smoke check: code unpacking, the near-tie
protocol, float tolerances, and stage-level comparisons between the CUDA path and the CPU oracle."""
from __future__ import annotations

import math

import numpy as np

REL_L2_TOL = 2e-3          # float outputs: relative L2 error
MAX_ABS_TOL = 1e-2         # float outputs: max abs error as a fraction of max |ref|


BYTE_CODES = 0x100         # flag of the C ABI: a `bits` value with it set stores one code per byte
PACKED6 = 0x200            # 6 | PACKED6: weight codes stored four to three bytes


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
    if bits == (6 | PACKED6):
        # code i in bits [6i, 6i + 6) of the row read as a little-endian bit string
        bits_le = ((q[:, :, None] >> np.arange(6, dtype=np.uint8)[None, None, :]) & 1).reshape(rows, n * 6)
        pad = (-bits_le.shape[1]) % 8
        bits_le = np.concatenate([bits_le, np.zeros((rows, pad), dtype=np.uint8)], axis=1)
        packed = np.packbits(bits_le, axis=1, bitorder="little")
        out[:, : packed.shape[1]] = packed
        return out
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


def check_ln_quant(rows, D, bits, bf16, seed=0, rms=False, eps=1e-6, pad_cols=0, want_sum=True, runs=1, inputs=None):
    """Runs the fused LN+quant kernel and compares its codes with the oracle's channel-wise codes.  With
    `runs` > 1 the launch is repeated and every launch has to write the bits of the first.  `inputs`, if given,
    is (x, gamma, beta, lo, hi) of a real workload instead of the stage-level generator's."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    x, gamma, beta, lo, hi = ln_case(rows, D, bf16, seed, rms, eps) if inputs is None else inputs
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
    g_dev, b_dev = torch.from_numpy(gamma_t).to(dev), torch.from_numpy(beta_t).to(dev)
    first = None
    for _ in range(runs):
        codes.fill_(0xEE)
        B.repq_ln_quant(xt, g_dev, b_dev, eps, s_t, z_t, bits, codes, row_sum,
                        B.REPQ_NORM_RMS if rms else B.REPQ_NORM_LAYERNORM)
        torch.cuda.synchronize()
        if first is None:
            first = codes.clone()
        assert torch.equal(codes, first), "launches differ"
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
    out32 = None
    if out_kind == "bf16":
        # the same product with float32 output: the bf16 output has to be its round-to-nearest-even, bit for bit
        out32 = torch.zeros(M, N, dtype=torch.float32, device=dev)
        d32 = B.gemm_desc(M, N, K, a_t, bits_a, float(s_a), int(z_a), w_t, bits_w, out32, s_w=s_w_t, z_w=z_w_t,
                          bias=bias_t, gelu=gelu, residual=res_t, acc_debug=None,
                          **{k: v for k, v in kw.items() if k not in ("out_kind",)})
        B.repq_qgemm(d32, ws)
        torch.cuda.synchronize()
        assert torch.equal(out32.to(torch.bfloat16), out), "bf16 output is not RNE(float32 output)"
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
            rel, mx = assert_float_close(out32.cpu().numpy(), v_ref, "qgemm (float32 value behind the bf16 output)")
            assert rel < 1e-5, rel
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
    if out_kind == "bf16":
        out32 = torch.zeros(B_ * Lq, D, dtype=torch.float32, device=dev)
        d.out_kind, d.out = B.REPQ_OUT_F32, out32.data_ptr()
        B.repq_pv(d)
        torch.cuda.synchronize()
        assert torch.equal(out32.to(torch.bfloat16), out), "bf16 output is not RNE(float32 output)"
        rel, _ = assert_float_close(out32.cpu().numpy(), O_ref, "pv (float32 value behind the bf16 output)")
        assert rel < 1e-5, rel
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
    y_dev = blk.forward(x)
    torch.cuda.synchronize()
    y = y_dev.float().cpu().numpy()
    assert np.all(np.isfinite(y))
    items = list(range(batch)) if sample_items is None else list(sample_items)
    rows = np.concatenate([np.arange(i * L, (i + 1) * L) for i in items])
    cfg = dict(w.cfg)
    cfg["B"] = len(items)
    w_s = dataclasses.replace(w, cfg=cfg, x=w.x[rows])
    ref = orc.block_forward(w_s)["y"]
    got = y[rows]
    if out_dtype == "bf16":
        # the bf16 output is the float32 output rounded to nearest even, bit for bit (rounding to bf16 alone costs
        # about 1.5e-3 of relative L2: the tolerance is spent on the float32 value)
        blk32 = QuantBlock(w, out_dtype=torch.float32, staged_attention=staged_attention)
        y32 = blk32.forward(x)
        torch.cuda.synchronize()
        assert torch.equal(y32.to(torch.bfloat16), y_dev), "bf16 block output is not RNE(float32 block output)"
        got = y32.cpu().numpy()[rows]
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


def check_attention(B_, H, Lq, Lk, dh, bits, bits_p, causal=False, out_kind="f32", out_bits=4 | BYTE_CODES, seed=0, s_p=1.0,
                    inputs=None, out_quant=None):
    """repq_attention (scores, Softmax, log-sqrt2 codes and P.V fused) against the oracle's chain of the same
    steps, all in float64 on the oracle's side.  A Softmax code whose pre-rounding value t sits on a rounding tie
    may legitimately differ by one (the near-tie protocol); such a flip changes the whole output row, so a row
    that holds near-ties is compared with every output the oracle gives with any subset of its tied codes moved
    to the other neighbour, and has to match one of them as strictly as an ordinary row matches its only one.

    `inputs`, if given, is (Qc, Kc, Vc, (s_q, z_q, s_k, z_k, s_v, z_v)): codes and quantizers of a real workload
    instead of the uniformly random ones; `out_quant` = (s_o, z_o) likewise replaces the output quantizer that is
    otherwise drawn from the output's percentiles."""
    import itertools
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    rng = np.random.default_rng(seed)
    D = H * dh
    nq = 1 << qb(bits)
    if inputs is None:
        Qc = rng.integers(0, nq, size=(B_ * Lq, D))
        Kc = rng.integers(0, nq, size=(B_ * Lk, D))
        Vc = rng.integers(0, nq, size=(B_ * Lk, D))
        z_q, z_k, z_v = (int(rng.integers(0, nq)) for _ in range(3))
        sig = (nq / 3.5) ** 2 * math.sqrt(dh)                 # rough std of sum (q - z_q)(k - z_k)
        s_q = s_k = math.sqrt(3.0 * math.sqrt(dh) / sig)      # logits with a standard deviation of about 3
        s_v = 0.05
    else:
        Qc, Kc, Vc, (s_q, z_q, s_k, z_k, s_v, z_v) = inputs
    # what the library is handed are float32 scales: the oracle takes the same numbers
    s_q, s_k, s_v, s_p = (float(np.float32(v)) for v in (s_q, s_k, s_v, s_p))
    alpha = float(np.float32(1.0 / math.sqrt(dh)))
    Qh, Kh, Vh = orc.dequant_uniform(Qc, s_q, z_q), orc.dequant_uniform(Kc, s_k, z_k), orc.dequant_uniform(Vc, s_v, z_v)
    shift = Lk - Lq
    valid = np.minimum(Lk, np.arange(Lq) + 1 + shift) if causal else np.full(Lq, Lk)
    O_ref = np.empty((B_ * Lq, D))
    absO = np.empty_like(O_ref)
    tie_rows = {}                                    # (b, h, i) -> list of (key j, the other neighbour of t)
    top = 2 ** qb(bits_p) - 1
    for b in range(B_):
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            S = Qh[b * Lq:(b + 1) * Lq, sl] @ Kh[b * Lk:(b + 1) * Lk, sl].T * alpha
            A = orc.softmax_rows(S, valid)
            p, t = orc.quant_logsqrt2(A, s_p, qb(bits_p))
            mask = np.arange(Lk)[None, :] < valid[:, None]
            tf = np.where(mask & np.isfinite(t), t, 0.25)
            m_row = np.where(mask, S, -np.inf).max(axis=1, keepdims=True)
            # width of a tie: float32 evaluation of t = 2 (log2 Z + log2 s) - 2 log2(e) (S - m) (2^-18 max(1, |t|), as
            # for the separate Softmax kernel) plus what the float32 scores carry into it.  S = float(integer sum) *
            # float(alpha s_q s_k): the rounding of the scale is common to S_i and m, so it is relative to S_i - m
            # (part of the |t| term); the rounding of m itself, 2^-24 |m|, enters t through 2 log2(e) = 2.9
            # The kernel may take its scores without the zero-point term of K, -z_k sum_c (q - z_q), which is common
            # to all keys of a row and drops out of the Softmax: its row maximum is then m + |that term| at most
            shift_row = np.abs(alpha * s_q * s_k * z_k * (Qc[b * Lq:(b + 1) * Lq, sl].astype(np.float64) - z_q).sum(axis=1, keepdims=True))
            delta = 2.0 ** -18 * np.maximum(1.0, np.abs(tf)) + 2.0 ** -22 * (np.abs(m_row) + shift_row)
            near = mask & (np.abs(tf - np.floor(tf) - 0.5) < delta) & (tf < min(top + 0.6, 40.0))   # a flip below a weight of 2^-20 is invisible
            for i, j in zip(*np.nonzero(near)):
                alt = int(np.clip(np.floor(tf[i, j]) + np.ceil(tf[i, j]) - np.rint(tf[i, j]), 0, top))
                if alt != int(p[i, j]):
                    tie_rows.setdefault((b, h, int(i)), []).append((int(j), alt))
            A_hat = np.where(mask, orc.dequant_logsqrt2(p, s_p), 0.0)
            O_ref[b * Lq:(b + 1) * Lq, sl] = A_hat @ Vh[b * Lk:(b + 1) * Lk, sl]
            absO[b * Lq:(b + 1) * Lq, sl] = A_hat @ np.abs(Vh[b * Lk:(b + 1) * Lk, sl])
            for (bb, hh, i), ties in tie_rows.items():
                if (bb, hh) == (b, h) and isinstance(ties, list):
                    # per tied key: what moving its code adds to the row's output
                    tie_rows[(bb, hh, i)] = [(j, (float(orc.dequant_logsqrt2(alt, s_p)) - A_hat[i, j]) * Vh[b * Lk + j, sl],
                                              abs(float(orc.dequant_logsqrt2(alt, s_p)) - A_hat[i, j]) * np.abs(Vh[b * Lk + j, sl]))
                                             for j, alt in ties]
                    tie_rows[(bb, hh, i)] = tuple(tie_rows[(bb, hh, i)])
    dev = torch.device("cuda:0")
    byte_bits = qb(bits) | BYTE_CODES
    q_t = torch.from_numpy(np.ascontiguousarray(Qc).astype(np.uint8)).to(dev)
    k_t = torch.from_numpy(np.ascontiguousarray(Kc).astype(np.uint8)).to(dev)
    v_t = torch.from_numpy(np.ascontiguousarray(Vc).astype(np.uint8)).to(dev)
    d = B.AttentionDesc()
    d.batch_outer, d.batch_inner, d.Lq, d.Lk, d.d_h, d.bits_qkv = B_, H, Lq, Lk, dh, byte_bits
    d.q_codes, d.ldq_bytes, d.q_stride_outer, d.q_stride_inner, d.s_q, d.z_q = q_t.data_ptr(), D, Lq * D, dh, s_q, z_q
    d.k_codes, d.ldk_bytes, d.k_stride_outer, d.k_stride_inner, d.s_k, d.z_k = k_t.data_ptr(), D, Lk * D, dh, s_k, z_k
    d.v_codes, d.ldv_bytes, d.v_stride_outer, d.v_stride_inner, d.s_v, d.z_v = v_t.data_ptr(), D, Lk * D, dh, s_v, z_v
    d.alpha, d.causal, d.bits_p, d.s_p = alpha, int(causal), bits_p, s_p

    def run(kind):
        row_sum = None
        if kind == "codes":
            ldo = B.code_row_bytes(D, out_bits)
            out = torch.full((B_ * Lq, ldo), 0xEE, dtype=torch.uint8, device=dev)
            d.out_kind, d.out_bits, d.out_scale, d.out_zero = B.REPQ_OUT_CODES, out_bits, float(s_o), int(z_o)
            d.ldo, d.o_stride_outer, d.o_stride_inner = ldo, Lq * ldo, (dh // 2 if out_bits == 4 else dh)
            row_sum = torch.zeros(B_ * Lq, dtype=torch.int32, device=dev)
            d.out_row_sum = row_sum.data_ptr()
        else:
            out = torch.zeros(B_ * Lq, D, dtype=torch.float32 if kind == "f32" else torch.bfloat16, device=dev)
            d.out_kind = B.REPQ_OUT_F32 if kind == "f32" else B.REPQ_OUT_BF16
            d.ldo, d.o_stride_outer, d.o_stride_inner = D, Lq * D, dh
            d.out_row_sum = None
        d.out = out.data_ptr()
        first = None
        for _ in range(3):                                   # repeated launches must agree bit for bit
            if row_sum is not None:
                row_sum.zero_()
            B.repq_attention(d)
            torch.cuda.synchronize()
            if first is None:
                first = out.clone()
            assert torch.equal(out, first), "launches differ"
        if qb(bits) == 4 and 0 <= z_q <= 15:
            # 4-bit Q / K: the score contraction ran on the 8-bit float type; the integer contraction must give the
            # same bits
            import os
            os.environ["REPQ_ATTENTION_INT_SCORES"] = "1"
            try:
                if row_sum is not None:
                    row_sum.zero_()
                B.repq_attention(d)
                torch.cuda.synchronize()
            finally:
                del os.environ["REPQ_ATTENTION_INT_SCORES"]
            assert torch.equal(out, first), "8-bit float scores and integer scores differ"
        assert B.repq_device_status() == 0
        return first, row_sum

    if out_kind == "codes":
        if out_quant is None:
            s_o, z_o = orc.uniform_scale_zero(np.percentile(O_ref, 1), np.percentile(O_ref, 99), qb(out_bits))
        else:
            s_o, z_o = out_quant
    out_t, row_sum = run(out_kind)
    if out_kind == "bf16":
        # the bf16 output is the float32 output rounded to nearest even, bit for bit; the float32 output is what
        # is compared with the oracle
        out32, _ = run("f32")
        assert torch.equal(out32.to(torch.bfloat16), out_t), "bf16 output is not RNE(float32 output)"
        out_t = out32

    def candidates(key):
        """Outputs of a row that holds near-ties: the oracle's, plus any subset of the tied codes moved."""
        b, h, i = key
        ties = tie_rows[key]
        base = O_ref[b * Lq + i, h * dh:(h + 1) * dh]
        base_abs = absO[b * Lq + i, h * dh:(h + 1) * dh]
        assert len(ties) <= 10, "a row with %d near-ties" % len(ties)
        for n in range(len(ties) + 1):
            for sub in itertools.combinations(ties, n):
                yield base + sum((dv for _, dv, _ in sub), np.zeros(dh)), base_abs + sum((da for _, _, da in sub), np.zeros(dh))

    tie_mask = np.zeros(B_ * Lq, dtype=bool)
    for (b, h, i) in tie_rows:
        tie_mask[b * Lq + i] = True
    keep = ~tie_mask
    n_tie = len(tie_rows)
    if out_kind == "codes":
        q_gpu = unpack_codes(out_t.cpu().numpy(), D, out_bits)

        def code_report(got, ref_rows, abs_rows):
            q_ref, t_ref = orc.quant_uniform(ref_rows, s_o, z_o, qb(out_bits))
            delta = 2.0 ** -17 * abs_rows / s_o + 2.0 ** -20 * np.abs(t_ref)
            return near_tie_report(got, q_ref, t_ref, delta)

        rep = code_report(q_gpu[keep], O_ref[keep], absO[keep])
        assert rep["bad"] == 0, rep
        for key in tie_rows:
            b, h, i = key
            got = q_gpu[b * Lq + i, h * dh:(h + 1) * dh]
            assert any(code_report(got, c, a)["bad"] == 0 for c, a in candidates(key)), ("tie row", key)
        # untied heads of a tied row
        for (b, h, i) in tie_rows:
            for h2 in range(H):
                if (b, h2, i) not in tie_rows:
                    s2 = slice(h2 * dh, (h2 + 1) * dh)
                    r = code_report(q_gpu[b * Lq + i, s2], O_ref[b * Lq + i, s2], absO[b * Lq + i, s2])
                    assert r["bad"] == 0, r
        assert np.array_equal(row_sum.cpu().numpy().astype(np.int64), q_gpu.sum(axis=1))
        rep["tie_rows"] = n_tie
        return rep
    got = out_t.double().cpu().numpy()
    rel, mx = assert_float_close(got[keep], O_ref[keep], "attention")
    assert rel < 1e-4, rel                               # exact operands, float32 sums: far inside the tolerance
    scale_all = np.abs(O_ref).max()
    for key in tie_rows:
        b, h, i = key
        g = got[b * Lq + i, h * dh:(h + 1) * dh]
        err = min(np.abs(g - c).max() / max(np.abs(c).max(), 1e-3 * scale_all) for c, _ in candidates(key))
        assert err < 1e-4, ("tie row", key, err)
    for (b, h, i) in tie_rows:
        for h2 in range(H):
            if (b, h2, i) not in tie_rows:
                s2 = slice(h2 * dh, (h2 + 1) * dh)
                ref = O_ref[b * Lq + i, s2]
                assert np.abs(got[b * Lq + i, s2] - ref).max() <= 1e-4 * max(np.abs(ref).max(), 1e-3 * scale_all)
    return dict(rel_l2=rel, max_abs=mx, tie_rows=n_tie)


def check_block_teacher_forced(name, **overrides):
    """Every stage of the block on the workload's own tensors, each fed the ORACLE's output of the stage before
    (`block_forward(keep=True)`), with the engine's folded parameters: LayerNorm codes, Q / K / V codes, attention
    codes, the residual stream, hidden codes and the block output are compared tensor by tensor, integer codes
    under the near-tie protocol.  One batch item."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from paper_2402_05628_b200.engine import QuantBlock
    from workloads import make_block_inputs

    w = make_block_inputs(name, batch=1, **overrides)
    cfg = w.cfg
    L, D, H, MLP = cfg["L"], cfg["D"], cfg["H"], cfg["MLP"]
    dh, M = D // H, cfg["L"]
    ba = cfg["bits_a"]
    ab = ba | BYTE_CODES
    llama = cfg.get("arch", "vit") == "llama"
    ref = orc.block_forward(w, keep=True)
    blk = QuantBlock(w, out_dtype=torch.float32)
    dev = blk.device
    norm_kind = B.REPQ_NORM_RMS if llama else B.REPQ_NORM_LAYERNORM
    rep = {}

    def dev_codes(q):
        return torch.from_numpy(np.ascontiguousarray(q).astype(np.uint8)).to(dev)

    def ln_stage(x_np, tag, g_dev, b_dev, s_t, z_t):
        x_t = torch.from_numpy(np.ascontiguousarray(x_np, dtype=np.float32)).to(dev).to(blk.act_dtype)
        codes = torch.full((M, D), 0xEE, dtype=torch.uint8, device=dev)
        rs = torch.zeros(M, dtype=torch.int32, device=dev)
        B.repq_ln_quant(x_t, g_dev, b_dev, cfg["eps"], s_t, z_t, ab, codes, rs, norm_kind)
        torch.cuda.synchronize()
        got = codes.cpu().numpy().astype(np.int64)
        h = blk.host[tag]
        t_cw = ref[tag + "_t"]
        t_lw = t_cw + (h["z"].astype(np.int64) - z_t)[None, :]
        r = near_tie_report(got, ref[tag + "_codes"], t_cw,
                            ln_delta(x_np, h["gamma_t"].astype(np.float64), s_t, t_lw, cfg["eps"], llama))
        assert r["bad"] == 0, (tag, r)
        assert r["mismatch"] <= max(2, 2e-4 * r["total"]), (tag, r)
        assert np.array_equal(rs.cpu().numpy().astype(np.int64), got.sum(axis=1))
        rep[tag] = r

    def linear_stage(a_codes, s_a, z_a, lin, N, **kw):
        a_t = dev_codes(a_codes)
        asum = torch.from_numpy(np.asarray(a_codes).sum(axis=1).astype(np.int32)).to(dev)
        return a_t, asum, dict(s_w=lin.s_w, z_w=lin.z_w, w_row_sum=lin.w_row_sum, bias=lin.bias, a_row_sum=asum, **kw)

    def run_gemm(d):
        ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 16), dtype=torch.uint8, device=dev)
        B.repq_qgemm(d, ws)
        torch.cuda.synchronize()
        assert B.repq_device_status() == 0

    def requant_report(got, name, mag):
        """Codes of a layer-wise quantizer against the oracle's; `mag` bounds the float32 terms behind the value."""
        lo, hi = w.bounds[name]
        s_o, _ = orc.uniform_scale_zero(lo, hi, ba)
        t = ref[name + "_t"]
        r = near_tie_report(got, ref[name + "_codes"], t, 2.0 ** -19 * mag / float(s_o) + 2.0 ** -20 * np.abs(t))
        assert r["bad"] == 0, (name, r)
        assert r["mismatch"] <= max(2, 2e-4 * r["total"]), (name, r)
        rep[name] = r

    # ---- LayerNorm 1 on x
    ln_stage(w.x, "ln1", blk.ln1_g, blk.ln1_b, blk.ln1_s, blk.ln1_z)

    # ---- QKV projection on the oracle's LayerNorm codes (rotary embedding in the epilogue for the LLaMA form)
    a_t, asum, kw = linear_stage(ref["ln1_codes"], blk.ln1_s, blk.ln1_z, blk.qkv, 3 * D)
    qkv = torch.full((M, 3 * D), 0xEE, dtype=torch.uint8, device=dev)
    quant = [blk.act_q[k] for k in ("q", "k", "v")]
    if llama:
        kw.update(rope=blk.rope, rope_period=L, rope_dim=dh, rope_groups=2)
    d = B.gemm_desc(M, 3 * D, D, a_t, ab, blk.ln1_s, blk.ln1_z, blk.qkv.codes, blk.bits_w, qkv, out_kind=B.REPQ_OUT_CODES,
                    out_bits=ab, out_scale=[q[0] for q in quant], out_zero=[q[1] for q in quant], **kw)
    run_gemm(d)
    got = qkv.cpu().numpy().astype(np.int64)
    b_t = blk.qkv.bias.cpu().numpy().astype(np.float64)
    for g, name in enumerate(("q", "k", "v")):
        s_o, _ = orc.uniform_scale_zero(*w.bounds[name], ba)
        v = ref[name + "_t"] * float(s_o)                           # the value the quantizer saw
        if llama and name != "v":                                   # a rotation keeps the length of a pair
            pair = np.sqrt(v[:, 0::2] ** 2 + v[:, 1::2] ** 2)
            v = np.repeat(pair, 2, axis=1)
            bias = np.abs(b_t[g * D:(g + 1) * D])
            bias = np.repeat(np.maximum(bias[0::2], bias[1::2]), 2)
            mag = 2.0 * (np.abs(v) + bias[None, :])
        else:
            mag = np.abs(v) + np.abs(b_t[g * D:(g + 1) * D])[None, :]
        requant_report(got[:, g * D:(g + 1) * D], name, 2.0 * mag)

    # ---- fused attention on the oracle's Q, K, V codes
    quants = []
    for name in ("q", "k", "v"):
        s_, z_ = orc.uniform_scale_zero(*w.bounds[name], ba)
        quants += [float(s_), int(z_)]
    s_at, z_at = orc.uniform_scale_zero(*w.bounds["attn"], ba)
    rep["attn"] = check_attention(1, H, L, L, dh, ab, cfg["bits_p"], causal=cfg["causal"], out_kind="codes", out_bits=ab,
                                  s_p=w.softmax_scale, inputs=(ref["q_codes"], ref["k_codes"], ref["v_codes"], tuple(quants)),
                                  out_quant=(float(s_at), int(z_at)))

    # ---- output projection on the oracle's attention codes, residual x: the residual stream X_bar
    s_a, z_a = blk.act_q["attn"]
    a_t, asum, kw = linear_stage(ref["attn_codes"], s_a, z_a, blk.proj, D)
    x_t = torch.from_numpy(np.ascontiguousarray(w.x)).to(dev).to(blk.act_dtype)
    xbar = torch.zeros(M, D, dtype=blk.act_dtype, device=dev)
    d = B.gemm_desc(M, D, D, a_t, ab, s_a, z_a, blk.proj.codes, blk.bits_w, xbar, residual=x_t,
                    out_kind=B.REPQ_OUT_BF16 if blk.act_dtype == torch.bfloat16 else B.REPQ_OUT_F32, **kw)
    run_gemm(d)
    got = xbar.float().cpu().numpy().astype(np.float64)
    xb = ref["x_bar"]
    if blk.act_dtype == torch.bfloat16:
        # RNE(float32 value) within one bf16 ulp of the oracle's rounded value; where the residual cancels the GEMM
        # value the float32 rounding of the two addends (2^-23 of each) remains in the small sum
        addends = np.abs(xb - w.x) + np.abs(w.x)
        assert np.all(np.abs(got - xb) <= np.abs(xb) * 2.0 ** -7 + addends * 2.0 ** -22 + 1e-30), "x_bar"
        rep["x_bar"] = float(np.mean(got != xb))
    else:
        rel, _ = assert_float_close(got, xb, "x_bar")
        assert rel < 1e-5, rel
        rep["x_bar"] = rel

    # ---- LayerNorm 2 on the oracle's residual stream
    ln_stage(xb, "ln2", blk.ln2_g, blk.ln2_b, blk.ln2_s, blk.ln2_z)

    # ---- fc1 on the oracle's LayerNorm-2 codes: GELU, or the gated product of the LLaMA form
    n_fc1 = 2 * MLP if llama else MLP
    a_t, asum, kw = linear_stage(ref["ln2_codes"], blk.ln2_s, blk.ln2_z, blk.fc1, n_fc1)
    hid = torch.full((M, MLP), 0xEE, dtype=torch.uint8, device=dev)
    s_h, z_h = blk.act_q["hidden"]
    d = B.gemm_desc(M, n_fc1, D, a_t, ab, blk.ln2_s, blk.ln2_z, blk.fc1.codes, blk.bits_w, hid, out_kind=B.REPQ_OUT_CODES,
                    out_bits=ab, out_scale=[s_h], out_zero=[z_h], gelu=not llama, glu=llama, **kw)
    run_gemm(d)
    pre = orc.linear_after_layernorm(ref["ln2_codes"], ref["ln2_s"], ref["ln2_z"], ref["ln2_rp"], ref["ln2_wcodes"],
                                     ref["ln2_sw"], ref["ln2_zw"])
    b_t = np.abs(ref["ln2_rp"]["b_t"])
    if llama:
        g_, u_ = pre[:, :MLP], pre[:, MLP:]
        dg = np.abs(g_) + b_t[None, :MLP]                  # float32 terms behind gate and up
        du = np.abs(u_) + b_t[None, MLP:]
        mag = 1.2 * dg * np.abs(u_) + np.abs(orc.silu(g_)) * du + 2.0 * np.abs(orc.silu(g_) * u_)      # ex2 / division approximations: 2^-20 of the product
    else:
        mag = 1.2 * (np.abs(pre) + b_t[None, :]) + np.abs(orc.gelu(pre))
    requant_report(hid.cpu().numpy().astype(np.int64), "hidden", 2.0 * mag)

    # ---- fc2 on the oracle's hidden codes, residual X_bar: the block output
    a_t, asum, kw = linear_stage(ref["hidden_codes"], s_h, z_h, blk.fc2, D)
    xb_t = torch.from_numpy(np.ascontiguousarray(xb, dtype=np.float32)).to(dev).to(blk.act_dtype)
    y = torch.zeros(M, D, dtype=torch.float32, device=dev)
    d = B.gemm_desc(M, D, MLP, a_t, ab, s_h, z_h, blk.fc2.codes, blk.bits_w, y, residual=xb_t, out_kind=B.REPQ_OUT_F32, **kw)
    run_gemm(d)
    rel, _ = assert_float_close(y.cpu().numpy(), ref["y"], "y")
    assert rel < 1e-5, rel
    rep["y"] = rel
    return rep


def check_qgemm_pair_step(M, N, K, bits, mode, out_kind="codes", seed=0, L=50, dh=32):
    """repq_qgemm with one of the two steps on neighbouring column pairs (LLaMA block form) against the oracle:
    mode "rope": the first two of three column ranges rotated by position m mod L (then Eq. 4 per range);
    mode "glu": columns (2i, 2i+1) = (gate, up), output silu(gate) * up (then Eq. 4)."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import gemm_codes

    rng = np.random.default_rng(seed)
    a, wq, s_a, z_a, s_w, z_w, bias = gemm_codes(rng, M, N, K, qb(bits), qb(bits))
    v_lin = orc.linear(orc.dequant_uniform(a, s_a, z_a), wq, s_w, z_w, bias)
    lin_mag = np.abs(v_lin - bias[None, :]) + np.abs(bias)[None, :]
    dev = torch.device("cuda:0")
    lda = B.code_row_bytes(K, bits)
    a_t = torch.from_numpy(pack_codes(a, bits, lda)).to(dev)
    w_t = torch.from_numpy(pack_codes(wq, bits, lda)).to(dev)
    s_w_t, z_w_t, bias_t = (torch.from_numpy(v).to(dev) for v in (s_w, z_w, bias))
    kw = dict(s_w=s_w_t, z_w=z_w_t, bias=bias_t)
    if mode == "rope":
        gw = N // 3
        H = gw // dh
        assert H * dh == gw and M % L == 0
        table = torch.from_numpy(B.repq_rope_table(L, dh, 10000.0)).to(dev)
        v_ref = v_lin.copy()
        mag = lin_mag.copy()
        for g in range(2):
            sl = slice(g * gw, (g + 1) * gw)
            v_ref[:, sl] = orc.rope(v_lin[:, sl], M // L, L, H, 10000.0)
            pm = np.sqrt(lin_mag[:, sl][:, 0::2] ** 2 + lin_mag[:, sl][:, 1::2] ** 2)
            mag[:, sl] = 2.0 * np.repeat(pm, 2, axis=1)
        kw.update(rope=table, rope_period=L, rope_dim=dh, rope_groups=2)
        n_out, groups = N, 3
    else:
        g_, u_ = v_lin[:, 0::2], v_lin[:, 1::2]
        v_ref = orc.silu(g_) * u_
        mag = 1.2 * lin_mag[:, 0::2] * np.abs(u_) + np.abs(orc.silu(g_)) * lin_mag[:, 1::2] + 2.0 * np.abs(v_ref)
        kw.update(glu=True)
        n_out, groups = N // 2, 1
    if out_kind == "codes":
        ob = qb(bits) | BYTE_CODES
        gw_o = n_out // groups
        lo = [np.percentile(v_ref[:, g * gw_o:(g + 1) * gw_o], 1) for g in range(groups)]
        hi = [np.percentile(v_ref[:, g * gw_o:(g + 1) * gw_o], 99) for g in range(groups)]
        s_o, z_o = orc.uniform_scale_zero(np.array(lo), np.array(hi), qb(bits))
        out = torch.full((M, B.code_row_bytes(n_out, ob)), 0xEE, dtype=torch.uint8, device=dev)
        rs = torch.zeros(M, dtype=torch.int32, device=dev)
        kw.update(out_kind=B.REPQ_OUT_CODES, out_bits=ob, out_scale=[float(v) for v in s_o], out_zero=[int(v) for v in z_o],
                  out_row_sum=rs)
    else:
        out = torch.zeros(M, n_out, dtype=torch.float32, device=dev)
        if mode == "rope":
            kw.update(out_scale=[1.0, 1.0, 1.0], out_zero=[0, 0, 0])          # three ranges: the first two are rotated
    d = B.gemm_desc(M, N, K, a_t, bits, float(s_a), int(z_a), w_t, bits, out, **kw)
    ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 16), dtype=torch.uint8, device=dev)
    B.repq_qgemm(d, ws)
    torch.cuda.synchronize()
    assert B.repq_device_status() == 0
    if out_kind != "codes":
        rel, mx = assert_float_close(out.cpu().numpy(), v_ref, "qgemm " + mode)
        assert rel < 2e-6, rel
        return dict(rel_l2=rel)
    q_gpu = out.cpu().numpy()[:, :n_out].astype(np.int64)
    rep = dict(total=0, mismatch=0, excused=0, bad=0)
    for g in range(groups):
        sl = slice(g * gw_o, (g + 1) * gw_o)
        q_ref, t_ref = orc.quant_uniform(v_ref[:, sl], s_o[g], z_o[g], qb(bits))
        r = near_tie_report(q_gpu[:, sl], q_ref, t_ref, 2.0 ** -19 * mag[:, sl] / s_o[g] + 2.0 ** -20 * np.abs(t_ref))
        for k in rep:
            rep[k] += r[k]
    assert rep["bad"] == 0, rep
    assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep
    assert np.array_equal(rs.cpu().numpy().astype(np.int64), q_gpu.sum(axis=1))
    return rep


def check_qgemm_repeated(M, N, K, bits, residual, out_kind, runs=12, seed=0):
    """A GEMM with a residual on dense random data, launched `runs` times: every launch reproduces the oracle and
    the first launch bit for bit (the residual boxes are refilled by bulk copies right after they are read)."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import gemm_codes, to_bf16_grid

    rng = np.random.default_rng(seed)
    b = bits | BYTE_CODES
    a, wq, s_a, z_a, s_w, z_w, bias = gemm_codes(rng, M, N, K, bits, bits)
    res = rng.normal(0, 1.0, size=(M, N)).astype(np.float32)
    if residual == "bf16":
        res = to_bf16_grid(res)
    v_ref = orc.linear(orc.dequant_uniform(a, s_a, z_a), wq, s_w, z_w, bias) + res
    dev = torch.device("cuda:0")
    a_t = torch.from_numpy(a.astype(np.uint8)).to(dev)
    w_t = torch.from_numpy(wq.astype(np.uint8)).to(dev)
    res_t = torch.from_numpy(res).to(dev)
    if residual == "bf16":
        res_t = res_t.to(torch.bfloat16)
    s_w_t, z_w_t, bias_t = (torch.from_numpy(v).to(dev) for v in (s_w, z_w, bias))
    out = torch.zeros(M, N, dtype=torch.float32 if out_kind == "f32" else torch.bfloat16, device=dev)
    d = B.gemm_desc(M, N, K, a_t, b, float(s_a), int(z_a), w_t, b, out, s_w=s_w_t, z_w=z_w_t, bias=bias_t, residual=res_t,
                    out_kind=B.REPQ_OUT_F32 if out_kind == "f32" else B.REPQ_OUT_BF16)
    ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 16), dtype=torch.uint8, device=dev)
    first = None
    for _ in range(runs):
        out.zero_()
        B.repq_qgemm(d, ws)
        torch.cuda.synchronize()
        if first is None:
            first = out.clone()
            got = out.float().cpu().numpy()
            if out_kind == "f32":
                rel, _ = assert_float_close(got, v_ref, "qgemm + residual")
                assert rel < 1e-5, rel
            else:
                ref16 = orc.round_bf16(v_ref)
                addends = np.abs(v_ref - res) + np.abs(res)
                assert np.all(np.abs(got - ref16) <= np.abs(ref16) * 2.0 ** -7 + addends * 2.0 ** -22 + 1e-30)
        assert torch.equal(out, first), "launches differ"
    assert B.repq_device_status() == 0


def check_dual_clip(n, D, bits, seed=0, iters=100, alpha0=2.0, strided=False):
    """repq_dual_clip against the oracle's per-channel dual clipping on LayerNorm activations of the stage-level
    generator: learned bounds and the objective before / after.  Both sides work in float64; they differ in the
    order of the sums over tokens, so a value that sits on a rounding tie to within round-off may steer one step of
    one channel differently: the bounds are compared to 1e-6 of the channel's range."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import affine_params, channel_profile, ln_inputs

    rng = np.random.default_rng(seed)
    c, shift = channel_profile(rng, D, 1.0, 0.02, 20.0)
    gamma, beta = affine_params(rng, D)
    X1 = orc.layernorm(ln_inputs(rng, n, c, shift, False), gamma, beta, 1e-6).astype(np.float32)
    ref = orc.dual_clip(X1, bits, iters=iters, lr=0.01, alpha0=alpha0)
    dev = torch.device("cuda:0")
    if strided:
        buf = torch.zeros(n, D + 5, dtype=torch.float32, device=dev)
        buf[:, :D] = torch.from_numpy(X1).to(dev)
        x_t = buf[:, :D]
    else:
        x_t = torch.from_numpy(X1).to(dev)
    lo = torch.full((D,), float("nan"), device=dev)
    hi = torch.full((D,), float("nan"), device=dev)
    loss = torch.zeros(2 * D, dtype=torch.float64, device=dev)
    B.repq_dual_clip(x_t, bits, lo, hi, loss, iters=iters, lr=0.01, alpha0=alpha0)
    torch.cuda.synchronize()
    rng_ch = X1.max(axis=0).astype(np.float64) - X1.min(axis=0)
    assert np.all(np.abs(lo.cpu().numpy() - ref["x_low"]) <= 1e-6 * rng_ch + 1e-7 * np.abs(ref["x_low"])), "x_low"
    assert np.all(np.abs(hi.cpu().numpy() - ref["x_up"]) <= 1e-6 * rng_ch + 1e-7 * np.abs(ref["x_up"])), "x_up"
    got = loss.cpu().numpy()
    assert np.allclose(got[:D], ref["loss0"], rtol=1e-9), "objective before the first step"
    assert np.allclose(got[D:], ref["loss"], rtol=1e-5), "objective with the learned bounds"
    return dict(loss0=float(ref["loss0"].sum()), loss=float(ref["loss"].sum()))


def check_calibration(name, batch, alpha0=2.0, **overrides):
    """The calibration pipeline on the GPU path (dual clipping, percentile calibration, every layer's input taken
    behind the layers already quantized) against the oracle's: the bounds found, then the block run with the
    GPU-calibrated bounds against the oracle block on the same bounds."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200.engine import QuantBlock, calibrate_block
    from workloads import make_block_inputs

    w = make_block_inputs(name, batch=batch, **overrides)
    ref = orc.block_forward(w, calibrate=dict(alpha0=alpha0))
    w_cal = calibrate_block(w, alpha0=alpha0)
    # LayerNorm bounds: to 1e-4 of the channel's range (float32 activations against float64, sums in another order)
    for tag in ("ln1", "ln2"):
        lo_r, hi_r = ref[tag + "_lo"].astype(np.float64), ref[tag + "_hi"].astype(np.float64)
        lo_g, hi_g = getattr(w_cal, tag + "_lo").astype(np.float64), getattr(w_cal, tag + "_hi").astype(np.float64)
        rng_ch = hi_r - lo_r
        frac_ok = np.mean((np.abs(lo_g - lo_r) <= 1e-4 * rng_ch) & (np.abs(hi_g - hi_r) <= 1e-4 * rng_ch))
        assert frac_ok >= 0.99, (tag, frac_ok)          # a rounding decision on a tie may steer one channel's steps apart
        assert np.all(np.abs(lo_g - lo_r) <= 2e-2 * rng_ch) and np.all(np.abs(hi_g - hi_r) <= 2e-2 * rng_ch), tag
    for key, (lo_r, hi_r) in ref["bounds"].items():
        lo_g, hi_g = w_cal.bounds[key]
        width = float(hi_r) - float(lo_r)
        assert abs(float(lo_g) - float(lo_r)) <= 2e-3 * width and abs(float(hi_g) - float(hi_r)) <= 2e-3 * width, (key, lo_g, lo_r, hi_g, hi_r)
    # the calibrated block: CUDA path against the oracle, both on the bounds the GPU pipeline found
    blk = QuantBlock(w_cal, out_dtype=torch.float32)
    x = torch.from_numpy(w.x).to(blk.device).to(blk.act_dtype)
    y = blk.forward(x)
    torch.cuda.synchronize()
    return assert_float_close(y.cpu().numpy(), orc.block_forward(w_cal)["y"], "calibrated block %s" % name)


# ------------------------------------------------------------------------------------------ sweep sizes, sampled

def check_ln_quant_sampled(rows, D, bits, n_sample=96, seed=4):
    """The fused LN+quant kernel at a sweep size (the launch the benchmark times), the oracle on sampled rows."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import affine_params, channel_profile, ln_calibration_bounds, ln_inputs

    rng = np.random.default_rng(seed)
    c, shift = channel_profile(rng, D, 1.0, 0.01, 50.0)
    gamma, beta = affine_params(rng, D)
    lo, hi = ln_calibration_bounds(ln_inputs(rng, 2048, c, shift, True), gamma, beta, 1e-6)
    x = ln_inputs(rng, rows, c, shift, True)
    s, z = orc.uniform_scale_zero(lo, hi, qb(bits))
    gamma_t, beta_t, s_t, z_t, _, _ = B.repq_fold_ln(gamma, beta, s.astype(np.float32), z.astype(np.int32),
                                                     np.zeros((1, D), dtype=np.float32), None)
    dev = torch.device("cuda:0")
    xt = torch.from_numpy(x).to(dev).to(torch.bfloat16)
    codes = torch.empty(rows, B.code_row_bytes(D, bits), dtype=torch.uint8, device=dev)
    rs = torch.empty(rows, dtype=torch.int32, device=dev)
    B.repq_ln_quant(xt, torch.from_numpy(gamma_t).to(dev), torch.from_numpy(beta_t).to(dev), 1e-6, s_t, z_t, bits, codes, rs)
    torch.cuda.synchronize()
    pick = np.unique(np.concatenate([[0, rows - 1], rng.integers(0, rows, n_sample)]))
    xs = x[pick]
    q_ref, t_cw = orc.quant_uniform(orc.layernorm(xs, gamma, beta, 1e-6), s[None, :], z[None, :], qb(bits))
    q_gpu = unpack_codes(codes[torch.from_numpy(pick).to(dev)].cpu().numpy(), D, bits)
    rep = near_tie_report(q_gpu, q_ref, t_cw, ln_delta(xs, gamma_t.astype(np.float64), s_t, t_cw + (z - z_t)[None, :], 1e-6, False))
    assert rep["bad"] == 0, rep
    assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep
    assert np.array_equal(rs.cpu().numpy()[pick].astype(np.int64), q_gpu.sum(axis=1))
    return rep


def check_softmax_log2_sampled(rows, L, bits, n_sample=64, seed=4):
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B
    from workloads.kernels import softmax_logits

    rng = np.random.default_rng(seed)
    # rows of the generator are independent: a block of distinct rows is tiled to the sweep's row count
    base = softmax_logits(rng, 1024, L)
    reps = (rows + 1023) // 1024
    dev = torch.device("cuda:0")
    ld = (L + 3) // 4 * 4
    buf = torch.zeros(1024, ld, dtype=torch.float32, device=dev)
    buf[:, :L] = torch.from_numpy(base).to(dev)
    S = buf.repeat(reps, 1)[:rows].contiguous()
    ldc = max(B.code_row_bytes(L, bits), (L + 7) // 8 * (4 if bits == 4 else 8))
    codes = torch.empty(rows, ldc, dtype=torch.uint8, device=dev)
    B.repq_softmax_log2(S, L, 1.0, bits, codes)
    torch.cuda.synchronize()
    pick = np.unique(np.concatenate([[0, rows - 1], rng.integers(0, rows, n_sample)]))
    q_ref, t_ref = orc.quant_logsqrt2(orc.softmax_rows(base[pick % 1024].astype(np.float64)), 1.0, qb(bits))
    q_gpu = unpack_codes(codes[torch.from_numpy(pick).to(dev)].cpu().numpy(), L, bits)
    delta = 2.0 ** -18 * np.maximum(1.0, np.abs(np.where(np.isfinite(t_ref), t_ref, 0.0)))
    rep = near_tie_report(q_gpu, q_ref, t_ref, delta)
    assert rep["bad"] == 0, rep
    assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep
    return rep


def check_qgemm_sampled(M, N, K, qbits, out_kind, n_sample=24, seed=4, weights="bytes"):  # weights: "bytes" | "packed"
    """repq_qgemm at a sweep size with the operand formats the benchmark times, the oracle on sampled rows."""
    import torch
    from oracle import repq_oracle as orc
    from paper_2402_05628_b200 import binding as B

    rng = np.random.default_rng(seed)
    bits = qbits | BYTE_CODES
    bits_w = (qbits | PACKED6 if qbits == 6 else qbits) if weights == "packed" else bits
    a = rng.integers(0, 1 << qbits, size=(M, K), dtype=np.uint8)
    wq = rng.integers(0, 1 << qbits, size=(N, K), dtype=np.uint8)
    s_a, z_a = np.float32(0.07), int(rng.integers(0, 1 << qbits))
    s_w = rng.uniform(0.001, 0.01, size=N).astype(np.float32)
    z_w = rng.integers(0, 1 << qbits, size=N, dtype=np.int32)
    bias = rng.normal(0.0, 0.02, size=N).astype(np.float32)
    dev = torch.device("cuda:0")
    a_t = torch.from_numpy(a).to(dev)
    w_t = torch.from_numpy(pack_codes(wq, bits_w, B.code_row_bytes(K, bits_w)) if weights == "packed" else wq).to(dev)
    s_w_t, z_w_t, bias_t = (torch.from_numpy(v).to(dev) for v in (s_w, z_w, bias))
    pick = np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, n_sample)]))
    v_ref = orc.linear(orc.dequant_uniform(a[pick], s_a, z_a), wq, s_w, z_w, bias)
    kw = {}
    if out_kind == "codes":
        s_o, z_o = orc.uniform_scale_zero(np.percentile(v_ref, 1), np.percentile(v_ref, 99), qbits)
        out = torch.empty(M, N, dtype=torch.uint8, device=dev)
        kw = dict(out_kind=B.REPQ_OUT_CODES, out_bits=bits, out_scale=[float(s_o)], out_zero=[int(z_o)])
    else:
        out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        kw = dict(out_kind=B.REPQ_OUT_BF16)
    d = B.gemm_desc(M, N, K, a_t, bits, float(s_a), z_a, w_t, bits_w, out, s_w=s_w_t, z_w=z_w_t, bias=bias_t, **kw)
    ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 16), dtype=torch.uint8, device=dev)
    B.repq_qgemm(d, ws)
    torch.cuda.synchronize()
    assert B.repq_device_status() == 0
    got = out[torch.from_numpy(pick).to(dev)]
    if out_kind == "codes":
        q_ref, t_ref = orc.quant_uniform(v_ref, s_o, z_o, qbits)
        mag = np.abs(v_ref - bias[None, :]) + np.abs(bias)[None, :] + np.abs(v_ref)
        rep = near_tie_report(got.cpu().numpy().astype(np.int64), q_ref, t_ref, 2.0 ** -19 * mag / s_o + 2.0 ** -20 * np.abs(t_ref))
        assert rep["bad"] == 0, rep
        assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep
        return rep
    ref16 = orc.round_bf16(v_ref)
    g = got.float().cpu().numpy()
    assert np.all(np.abs(g - ref16) <= np.abs(ref16) * 2.0 ** -7 + 1e-30)
    return dict(rel_l2=float_errors(g, v_ref)[0])
