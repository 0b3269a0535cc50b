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
                 weight_storage: str = "packed"):
        """weight_storage: "packed" keeps 4-bit weight codes two per byte in device memory (the GEMM expands the
        tiles in shared memory); "bytes" keeps one code per byte, the tensor-core operand format."""
        assert weight_storage in ("packed", "bytes")
        self.weight_storage = weight_storage
        self.staged_attention = bool(staged_attention)
        cfg = w.cfg
        self.cfg = cfg
        dev = torch.device(device)
        self.device = dev
        ba = cfg["bits_a"]
        bw = self.bits_w = cfg["bits_w"] if weight_storage == "packed" else cfg["bits_w"] | B.REPQ_BYTE_CODES
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
