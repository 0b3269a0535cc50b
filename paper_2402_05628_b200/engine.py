"""Prepares a quantized transformer block for the library and runs it.

Preparation is one-time and uses only the library's host entry points: Eq. 6 quantizer parameters
from clipping bounds, the LayerNorm scale reparameterization (Eqs. 10-14) and channel-wise weight
packing.  The forward pass is a single `repq_block_forward` call.  This module only moves arrays
between numpy, torch and the C ABI.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as B


@dataclasses.dataclass
class PreparedLinear:
    codes: torch.Tensor
    s_w: torch.Tensor
    z_w: torch.Tensor
    w_row_sum: torch.Tensor
    bias: torch.Tensor

    def params(self) -> B.LinearParams:
        p = B.LinearParams()
        p.w_codes, p.ldw_bytes = self.codes.data_ptr(), self.codes.stride(0)
        p.s_w, p.z_w = self.s_w.data_ptr(), self.z_w.data_ptr()
        p.w_row_sum, p.bias = self.w_row_sum.data_ptr(), self.bias.data_ptr()
        return p


def _pack_linear(W: np.ndarray, bias: np.ndarray, bits_w: int, dev) -> PreparedLinear:
    codes, s_w, z_w, wsum = B.repq_pack_weights(W, bits_w)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    return PreparedLinear(t(codes), t(s_w), t(z_w), t(wsum), t(np.asarray(bias, dtype=np.float32)))


class QuantBlock:
    """Device-resident parameters of one block plus its workspace; `forward` runs the hot path."""

    def __init__(self, w, device="cuda:0", out_dtype: Optional[torch.dtype] = None, staged_attention: bool = False,
                 weight_storage: str = "bytes"):
        """weight_storage: "packed" keeps 4-bit weight codes two per byte and 6-bit codes four to three bytes in device
        memory (the GEMM expands the tiles in shared memory); "bytes" keeps one code per byte, the tensor-core operand
        format."""
        assert weight_storage in ("packed", "bytes")
        self.weight_storage = weight_storage
        self.staged_attention = bool(staged_attention)
        cfg = w.cfg
        self.cfg = cfg
        dev = torch.device(device)
        self.device = dev
        ba = cfg["bits_a"]
        if weight_storage == "packed":
            bw = cfg["bits_w"] | B.REPQ_PACKED6 if cfg["bits_w"] == 6 else cfg["bits_w"]
        else:
            bw = cfg["bits_w"] | B.REPQ_BYTE_CODES
        self.bits_w = bw
        self.host: Dict[str, object] = {}

        def fold(gamma, beta, lo, hi, W, b, tag):
            s, z = B.repq_scale_zero_from_bounds(lo, hi, ba)
            g_t, b_t, s_t, z_t, W_t, bias_t = B.repq_fold_ln(gamma, beta, s, z, W, b)
            self.host[tag] = dict(s=s, z=z, gamma_t=g_t, beta_t=b_t, s_t=s_t, z_t=z_t)
            return (torch.from_numpy(g_t).to(dev), torch.from_numpy(b_t).to(dev), s_t, z_t,
                    _pack_linear(W_t, bias_t, bw, dev))

        self.llama = cfg.get("arch", "vit") == "llama"
        w_fc1, b_fc1 = w.w_fc1, w.b_fc1
        if self.llama:
            # gated MLP: the library takes gate_i and up_i as neighbouring weight rows (2i, 2i+1)
            mlp = cfg["MLP"]
            order = np.stack([np.arange(mlp), mlp + np.arange(mlp)], axis=1).reshape(-1)
            w_fc1, b_fc1 = w.w_fc1[order], w.b_fc1[order]
        self.ln1_g, self.ln1_b, self.ln1_s, self.ln1_z, self.qkv = fold(
            w.ln1_gamma, w.ln1_beta, w.ln1_lo, w.ln1_hi, w.w_qkv, w.b_qkv, "ln1")
        self.ln2_g, self.ln2_b, self.ln2_s, self.ln2_z, self.fc1 = fold(
            w.ln2_gamma, w.ln2_beta, w.ln2_lo, w.ln2_hi, w_fc1, b_fc1, "ln2")
        self.rope = None
        if self.llama:
            self.rope = torch.from_numpy(B.repq_rope_table(cfg["L"], cfg["D"] // cfg["H"], cfg.get("rope_base", 10000.0))).to(dev)
        self.proj = _pack_linear(w.w_proj, w.b_proj, bw, dev)
        self.fc2 = _pack_linear(w.w_fc2, w.b_fc2, bw, dev)
        self.act_q = {}
        for key in ("q", "k", "v", "attn", "hidden"):
            lo, hi = w.bounds[key]
            s, z = B.repq_scale_zero_from_bounds(np.float32(lo), np.float32(hi), ba)
            self.act_q[key] = (float(s[0]), int(z[0]))

        self.act_dtype = torch.float32 if cfg["act"] == "f32" else torch.bfloat16
        self.out_dtype = out_dtype or self.act_dtype
        self.softmax_s = float(w.softmax_scale)
        self._ws: Optional[torch.Tensor] = None
        self._staging = None
        self._batch = None

    def desc(self, batch: int) -> B.BlockDesc:
        c = self.cfg
        d = B.BlockDesc()
        d.batch, d.seq, d.dim, d.heads, d.mlp = batch, c["L"], c["D"], c["H"], c["MLP"]
        d.bits_a, d.bits_w, d.bits_p = c["bits_a"], self.bits_w, c["bits_p"]
        d.causal, d.eps = int(c["causal"]), c["eps"]
        d.norm_kind = B.REPQ_NORM_RMS if self.llama else B.REPQ_NORM_LAYERNORM
        d.rope = int(self.llama)
        d.mlp_kind = B.REPQ_MLP_SWIGLU if self.llama else B.REPQ_MLP_GELU
        d.act_dtype = B.REPQ_F32 if self.act_dtype == torch.float32 else B.REPQ_BF16
        d.out_dtype = B.REPQ_F32 if self.out_dtype == torch.float32 else B.REPQ_BF16
        d.staged_attention = int(self.staged_attention)
        return d

    def params(self) -> B.BlockParams:
        p = B.BlockParams()
        p.ln1_gamma_t, p.ln1_beta_t, p.ln1_s, p.ln1_z = self.ln1_g.data_ptr(), self.ln1_b.data_ptr(), self.ln1_s, self.ln1_z
        p.qkv = self.qkv.params()
        (p.s_q, p.z_q), (p.s_k, p.z_k), (p.s_v, p.z_v) = self.act_q["q"], self.act_q["k"], self.act_q["v"]
        p.softmax_s = self.softmax_s
        p.s_attn, p.z_attn = self.act_q["attn"]
        p.proj = self.proj.params()
        p.ln2_gamma_t, p.ln2_beta_t, p.ln2_s, p.ln2_z = self.ln2_g.data_ptr(), self.ln2_b.data_ptr(), self.ln2_s, self.ln2_z
        p.fc1 = self.fc1.params()
        p.s_hidden, p.z_hidden = self.act_q["hidden"]
        p.fc2 = self.fc2.params()
        p.rope_cos_sin = self.rope.data_ptr() if self.rope is not None else None
        return p

    def workspace(self, batch: int) -> torch.Tensor:
        if self._ws is None or self._batch != batch:
            n = B.repq_block_workspace_bytes(self.desc(batch))
            self._ws = torch.empty(n + 256, dtype=torch.uint8, device=self.device)
            off = (-self._ws.data_ptr()) % 256
            self._ws = self._ws[off:off + n]
            self._batch = batch
        return self._ws

    def forward(self, x: torch.Tensor, y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """x: [batch * seq, dim] on the device, dtype = activation dtype of the config."""
        c = self.cfg
        assert x.dtype == self.act_dtype and x.is_contiguous() and x.shape[1] == c["D"]
        batch = x.shape[0] // c["L"]
        assert batch * c["L"] == x.shape[0]
        if y is None:
            y = torch.empty(x.shape, dtype=self.out_dtype, device=x.device)
        B.repq_block_forward(self.desc(batch), self.params(), x, y, self.workspace(batch), stream)
        return y

    def forward_host(self, x_host: List[torch.Tensor], y_host: List[torch.Tensor], stream=None) -> None:
        """The block over batches held in (pinned) host memory: x_host[i] -> y_host[i], every tensor
        [batch * seq, dim].  Copies in, kernels and copies out of neighbouring batches overlap; y_host is valid
        once `stream` (default: the current stream) has completed."""
        c = self.cfg
        if not x_host:
            return
        rows = x_host[0].shape[0]
        batch = rows // c["L"]
        for t in x_host:
            assert t.dtype == self.act_dtype and t.is_contiguous() and tuple(t.shape) == (rows, c["D"]) and not t.is_cuda
        for t in y_host:
            assert t.dtype == self.out_dtype and t.is_contiguous() and tuple(t.shape) == (rows, c["D"]) and not t.is_cuda
        if self._staging is None or self._staging[0][0].shape[0] != rows:
            self._staging = ([torch.empty((rows, c["D"]), dtype=self.act_dtype, device=self.device) for _ in range(2)],
                             [torch.empty((rows, c["D"]), dtype=self.out_dtype, device=self.device) for _ in range(2)])
        B.repq_block_forward_host(self.desc(batch), self.params(), x_host, y_host, self._staging[0], self._staging[1],
                                  self.workspace(batch), stream)

    def forward_timed(self, x: torch.Tensor, y: torch.Tensor, stream=None) -> List[float]:
        """Same pass with per-stage CUDA-event timing (synchronises); returns milliseconds per stage."""
        batch = x.shape[0] // self.cfg["L"]
        return B.repq_block_forward_timed(self.desc(batch), self.params(), x, y, self.workspace(batch), stream)


def _percentile(t: torch.Tensor, pct: float) -> float:
    """Percentile with linear interpolation between order statistics (a sort: library call, host-side calibration)."""
    v, _ = torch.sort(t.reshape(-1).float())
    pos = (v.numel() - 1) * pct / 100.0
    i = int(pos)
    frac = pos - i
    lo = float(v[i])
    hi = float(v[min(i + 1, v.numel() - 1)])
    return lo + (hi - lo) * frac


def calibrate_block(w, device="cuda:0", alpha0: float = 0.0, iters: int = 100, lr: float = 0.01,
                    lo_pct: float = 0.1, hi_pct: float = 99.9):
    """Sequential pipeline of Algorithm 1 for one block on the calibration batch `w.x`, round-to-nearest weight
    quantization in GPTQ's place: every quantizer's bounds are found on the input that reaches it through the layers
    already quantized.  LayerNorm activations: full-precision normalisation (repq_layernorm), per-channel dual
    clipping (repq_dual_clip, Eqs. 18-20), scale reparameterization (repq_fold_ln).  Every other activation:
    percentile calibration on the float32 output of the quantized layer before it (repq_qgemm / repq_attention with
    float outputs).  Returns a copy of `w` whose clipping bounds are the calibrated ones; `QuantBlock` of that copy
    is the calibrated block.  This function only sequences library calls and sorts for the percentiles."""
    import dataclasses
    cfg = w.cfg
    dev = torch.device(device)
    L, D, H, MLP = cfg["L"], cfg["D"], cfg["H"], cfg["MLP"]
    dh = D // H
    ba = cfg["bits_a"]
    ab = ba | B.REPQ_BYTE_CODES
    bw = cfg["bits_w"]
    llama = cfg.get("arch", "vit") == "llama"
    norm_kind = B.REPQ_NORM_RMS if llama else B.REPQ_NORM_LAYERNORM
    act_dtype = torch.float32 if cfg["act"] == "f32" else torch.bfloat16
    x = torch.from_numpy(np.ascontiguousarray(w.x)).to(dev).to(act_dtype)
    M = x.shape[0]
    batch = M // L
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    bounds = {}

    def quantizer(name, values):
        lo, hi = np.float32(_percentile(values, lo_pct)), np.float32(_percentile(values, hi_pct))
        bounds[name] = (lo, hi)
        s, z = B.repq_scale_zero_from_bounds(lo, hi, ba)
        return float(s[0]), int(z[0])

    def after_norm(x_in, gamma, beta, W, b):
        """Dual clipping on the normalised calibration batch, fold, pack, and the LayerNorm codes of the batch."""
        X1 = torch.empty(M, D, dtype=torch.float32, device=dev)
        B.repq_layernorm(x_in, t(gamma), t(beta), cfg["eps"], X1, norm_kind)
        lo, hi = torch.empty(D, device=dev), torch.empty(D, device=dev)
        B.repq_dual_clip(X1, ba, lo, hi, None, iters=iters, lr=lr, alpha0=alpha0)
        lo, hi = lo.cpu().numpy(), hi.cpu().numpy()
        s, z = B.repq_scale_zero_from_bounds(lo, hi, ba)
        g_t, b_t, s_t, z_t, W_t, bias_t = B.repq_fold_ln(gamma, beta, s, z, W, b)
        lin = _pack_linear(W_t, bias_t, bw, dev)
        codes = torch.empty(M, D, dtype=torch.uint8, device=dev)
        rs = torch.empty(M, dtype=torch.int32, device=dev)
        B.repq_ln_quant(x_in, t(g_t), t(b_t), cfg["eps"], s_t, z_t, ab, codes, rs, norm_kind)
        return lo, hi, lin, codes, rs, s_t, z_t

    def gemm(a, s_a, z_a, asum, lin, N, K, out, **kw):
        d = B.gemm_desc(M, N, K, a, ab, s_a, z_a, lin.codes, bw, out, s_w=lin.s_w, z_w=lin.z_w, w_row_sum=lin.w_row_sum,
                        bias=lin.bias, a_row_sum=asum, **kw)
        ws = torch.empty(max(B.repq_qgemm_workspace_bytes(d), 16), dtype=torch.uint8, device=dev)
        B.repq_qgemm(d, ws)
        torch.cuda.synchronize()

    # ---- LayerNorm 1 -> QKV
    ln1_lo, ln1_hi, qkv, c1, rs1, s1, z1 = after_norm(x, w.ln1_gamma, w.ln1_beta, w.w_qkv, w.b_qkv)
    rope = None
    kw = {}
    if llama:
        rope = t(B.repq_rope_table(L, dh, cfg.get("rope_base", 10000.0)))
        kw = dict(rope=rope, rope_period=L, rope_dim=dh, rope_groups=2)
    qkv_f = torch.empty(M, 3 * D, dtype=torch.float32, device=dev)
    gemm(c1, s1, z1, rs1, qkv, 3 * D, D, qkv_f, out_scale=[1.0] * 3, out_zero=[0] * 3, **kw)
    quant = [quantizer(n, qkv_f[:, i * D:(i + 1) * D]) for i, n in enumerate(("q", "k", "v"))]
    qkv_c = torch.empty(M, 3 * D, dtype=torch.uint8, device=dev)
    gemm(c1, s1, z1, rs1, qkv, 3 * D, D, qkv_c, out_kind=B.REPQ_OUT_CODES, out_bits=ab, out_scale=[q[0] for q in quant],
         out_zero=[q[1] for q in quant], **kw)
    del qkv_f

    # ---- attention (float output for the calibration of its quantizer, then codes)
    a = B.AttentionDesc()
    a.batch_outer, a.batch_inner, a.Lq, a.Lk, a.d_h, a.bits_qkv = batch, H, L, L, dh, ab
    for i, n in enumerate("qkv"):
        setattr(a, n + "_codes", qkv_c.data_ptr() + i * D)
        setattr(a, "ld%s_bytes" % n, 3 * D)
        setattr(a, n + "_stride_outer", L * 3 * D)
        setattr(a, n + "_stride_inner", dh)
        setattr(a, "s_" + n, quant[i][0])
        setattr(a, "z_" + n, quant[i][1])
    a.alpha, a.causal, a.bits_p, a.s_p = 1.0 / float(np.sqrt(dh)), int(cfg["causal"]), cfg["bits_p"], float(w.softmax_scale)
    o_f = torch.empty(M, D, dtype=torch.float32, device=dev)
    a.out_kind, a.out, a.ldo, a.o_stride_outer, a.o_stride_inner = B.REPQ_OUT_F32, o_f.data_ptr(), D, L * D, dh
    B.repq_attention(a)
    torch.cuda.synchronize()
    s_at, z_at = quantizer("attn", o_f)
    o_c = torch.empty(M, D, dtype=torch.uint8, device=dev)
    rs_o = torch.zeros(M, dtype=torch.int32, device=dev)
    a.out_kind, a.out_bits, a.out_scale, a.out_zero = B.REPQ_OUT_CODES, ab, s_at, z_at
    a.out, a.out_row_sum = o_c.data_ptr(), rs_o.data_ptr()
    B.repq_attention(a)
    torch.cuda.synchronize()

    # ---- output projection + residual: the residual stream
    proj = _pack_linear(w.w_proj, w.b_proj, bw, dev)
    xbar = torch.empty(M, D, dtype=act_dtype, device=dev)
    gemm(o_c, s_at, z_at, rs_o, proj, D, D, xbar, residual=x,
         out_kind=B.REPQ_OUT_F32 if act_dtype == torch.float32 else B.REPQ_OUT_BF16)

    # ---- LayerNorm 2 -> fc1 -> activation
    w_fc1, b_fc1 = w.w_fc1, w.b_fc1
    if llama:
        order = np.stack([np.arange(MLP), MLP + np.arange(MLP)], axis=1).reshape(-1)
        w_fc1, b_fc1 = w.w_fc1[order], w.b_fc1[order]
    ln2_lo, ln2_hi, fc1, c2, rs2, s2, z2 = after_norm(xbar, w.ln2_gamma, w.ln2_beta, w_fc1, b_fc1)
    h_f = torch.empty(M, MLP, dtype=torch.float32, device=dev)
    gemm(c2, s2, z2, rs2, fc1, 2 * MLP if llama else MLP, D, h_f, gelu=not llama, glu=llama)
    quantizer("hidden", h_f)
    assert B.repq_device_status() == 0
    return dataclasses.replace(w, ln1_lo=ln1_lo, ln1_hi=ln1_hi, ln2_lo=ln2_lo, ln2_hi=ln2_hi, bounds=bounds)
