"""ctypes binding of librepq.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors (device memory and streams come from PyTorch); every computation happens
inside the library's CUDA kernels.  A missing library is a hard error: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librepq.so")

REPQ_OK = 0
REPQ_INVALID_ARG, REPQ_UNSUPPORTED, REPQ_ALIGNMENT, REPQ_WORKSPACE_TOO_SMALL, REPQ_CUDA_ERROR, REPQ_TIMEOUT = 1, 2, 3, 4, 5, 6
REPQ_F32, REPQ_BF16 = 0, 1
REPQ_NORM_LAYERNORM, REPQ_NORM_RMS = 0, 1
REPQ_OUT_F32, REPQ_OUT_BF16, REPQ_OUT_CODES = 0, 1, 2
REPQ_MAX_OUT_GROUPS = 4
REPQ_BYTE_CODES = 0x100
REPQ_PACKED6 = 0x200          # 6 | REPQ_PACKED6: weight codes, four in three bytes

EXPORTS = (
    "repq_last_error", "repq_abi_version", "repq_scale_zero_from_bounds", "repq_fold_ln",
    "repq_pack_weights", "repq_ln_quant", "repq_qgemm_workspace_bytes", "repq_qgemm",
    "repq_softmax_log2", "repq_pv", "repq_block_workspace_bytes", "repq_block_forward",
    "repq_device_status", "repq_block_forward_timed", "repq_launch_count",
    "repq_block_forward_static", "repq_attention", "repq_block_forward_host", "repq_rope_table",
    "repq_bounded_wait_selftest", "repq_dual_clip", "repq_layernorm",
)
REPQ_MLP_GELU, REPQ_MLP_SWIGLU = 0, 1
REPQ_STATIC_WORKSPACE_BYTES = 8 << 20
REPQ_BLOCK_STAGES = 9
BLOCK_STAGE_NAMES = ("ln1", "qkv", "scores", "softmax", "pv", "proj", "ln2", "fc1", "fc2")


class RepqError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("repq status %d: %s" % (status, message))
        self.status = status


class GemmDesc(C.Structure):
    _fields_ = [
        ("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32),
        ("batch_outer", C.c_int32), ("batch_inner", C.c_int32),
        ("a_codes", C.c_void_p), ("bits_a", C.c_int32),
        ("lda_bytes", C.c_int64), ("a_stride_outer", C.c_int64), ("a_stride_inner", C.c_int64),
        ("s_a", C.c_float), ("z_a", C.c_int32), ("a_row_sum", C.c_void_p),
        ("w_codes", C.c_void_p), ("bits_w", C.c_int32),
        ("ldw_bytes", C.c_int64), ("w_stride_outer", C.c_int64), ("w_stride_inner", C.c_int64),
        ("s_w", C.c_void_p), ("z_w", C.c_void_p), ("s_w_scalar", C.c_float), ("z_w_scalar", C.c_int32),
        ("w_row_sum", C.c_void_p), ("bias", C.c_void_p), ("alpha", C.c_float),
        ("gelu", C.c_int32), ("residual", C.c_void_p), ("residual_dtype", C.c_int32),
        ("ld_residual", C.c_int64),
        ("out_kind", C.c_int32), ("out_bits", C.c_int32), ("out_groups", C.c_int32),
        ("out_scale", C.c_float * REPQ_MAX_OUT_GROUPS), ("out_zero", C.c_int32 * REPQ_MAX_OUT_GROUPS),
        ("out", C.c_void_p), ("ldo", C.c_int64), ("o_stride_outer", C.c_int64), ("o_stride_inner", C.c_int64),
        ("out_row_sum", C.c_void_p), ("acc_debug", C.c_void_p), ("causal", C.c_int32),
        ("rope_cos_sin", C.c_void_p), ("rope_period", C.c_int32), ("rope_dim", C.c_int32), ("rope_groups", C.c_int32),
        ("glu", C.c_int32),
    ]


class PvDesc(C.Structure):
    _fields_ = [
        ("batch_outer", C.c_int32), ("batch_inner", C.c_int32), ("Lq", C.c_int32), ("Lk", C.c_int32),
        ("d_h", C.c_int32),
        ("p_codes", C.c_void_p), ("bits_p", C.c_int32), ("ldp_bytes", C.c_int64), ("p_stride_pair", C.c_int64),
        ("s_p", C.c_float),
        ("v_codes", C.c_void_p), ("bits_v", C.c_int32), ("ldv_bytes", C.c_int64),
        ("v_stride_outer", C.c_int64), ("v_stride_inner", C.c_int64), ("s_v", C.c_float), ("z_v", C.c_int32),
        ("causal", C.c_int32), ("out_kind", C.c_int32), ("out_bits", C.c_int32), ("out_scale", C.c_float),
        ("out_zero", C.c_int32), ("out", C.c_void_p), ("ldo", C.c_int64), ("o_stride_outer", C.c_int64),
        ("o_stride_inner", C.c_int64), ("out_row_sum", C.c_void_p),
    ]


class LinearParams(C.Structure):
    _fields_ = [("w_codes", C.c_void_p), ("ldw_bytes", C.c_int64), ("s_w", C.c_void_p), ("z_w", C.c_void_p),
                ("w_row_sum", C.c_void_p), ("bias", C.c_void_p)]


class BlockDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq", C.c_int32), ("dim", C.c_int32), ("heads", C.c_int32),
                ("mlp", C.c_int32), ("bits_a", C.c_int32), ("bits_w", C.c_int32), ("bits_p", C.c_int32),
                ("causal", C.c_int32), ("norm_kind", C.c_int32), ("eps", C.c_float),
                ("act_dtype", C.c_int32), ("out_dtype", C.c_int32), ("staged_attention", C.c_int32),
                ("rope", C.c_int32), ("mlp_kind", C.c_int32)]


class AttentionDesc(C.Structure):
    _fields_ = [
        ("batch_outer", C.c_int32), ("batch_inner", C.c_int32), ("Lq", C.c_int32), ("Lk", C.c_int32), ("d_h", C.c_int32),
        ("bits_qkv", C.c_int32),
        ("q_codes", C.c_void_p), ("ldq_bytes", C.c_int64), ("q_stride_outer", C.c_int64), ("q_stride_inner", C.c_int64),
        ("s_q", C.c_float), ("z_q", C.c_int32),
        ("k_codes", C.c_void_p), ("ldk_bytes", C.c_int64), ("k_stride_outer", C.c_int64), ("k_stride_inner", C.c_int64),
        ("s_k", C.c_float), ("z_k", C.c_int32),
        ("v_codes", C.c_void_p), ("ldv_bytes", C.c_int64), ("v_stride_outer", C.c_int64), ("v_stride_inner", C.c_int64),
        ("s_v", C.c_float), ("z_v", C.c_int32),
        ("alpha", C.c_float), ("causal", C.c_int32), ("bits_p", C.c_int32), ("s_p", C.c_float),
        ("out_kind", C.c_int32), ("out_bits", C.c_int32), ("out_scale", C.c_float), ("out_zero", C.c_int32),
        ("out", C.c_void_p), ("ldo", C.c_int64), ("o_stride_outer", C.c_int64), ("o_stride_inner", C.c_int64),
        ("out_row_sum", C.c_void_p),
    ]


class BlockParams(C.Structure):
    _fields_ = [
        ("ln1_gamma_t", C.c_void_p), ("ln1_beta_t", C.c_void_p), ("ln1_s", C.c_float), ("ln1_z", C.c_int32),
        ("qkv", LinearParams),
        ("s_q", C.c_float), ("s_k", C.c_float), ("s_v", C.c_float),
        ("z_q", C.c_int32), ("z_k", C.c_int32), ("z_v", C.c_int32),
        ("softmax_s", C.c_float), ("s_attn", C.c_float), ("z_attn", C.c_int32),
        ("proj", LinearParams),
        ("ln2_gamma_t", C.c_void_p), ("ln2_beta_t", C.c_void_p), ("ln2_s", C.c_float), ("ln2_z", C.c_int32),
        ("fc1", LinearParams), ("s_hidden", C.c_float), ("z_hidden", C.c_int32),
        ("fc2", LinearParams),
        ("rope_cos_sin", C.c_void_p),
    ]


_lib = None


def lib() -> C.CDLL:
    """Loads librepq.so; raises if it has not been built (there is no CPU or PyTorch fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("librepq.so is missing: build it with `python -m paper_2402_05628_b200.build` "
                              "(needs nvcc); the repq hot path has no fallback implementation")
        _lib = C.CDLL(LIB_PATH)
        _lib.repq_last_error.restype = C.c_size_t
        _lib.repq_last_error.argtypes = [C.c_char_p, C.c_size_t]
        _lib.repq_ln_quant.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int64, C.c_void_p, C.c_void_p,
                                       C.c_float, C.c_int, C.c_float, C.c_int, C.c_int, C.c_void_p, C.c_int64,
                                       C.c_void_p, C.c_void_p]
        _lib.repq_softmax_log2.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int64, C.c_float, C.c_int,
                                           C.c_int, C.c_float, C.c_int, C.c_void_p, C.c_int64, C.c_void_p]
        _lib.repq_qgemm_workspace_bytes.argtypes = [C.POINTER(GemmDesc), C.POINTER(C.c_size_t)]
        _lib.repq_qgemm.argtypes = [C.POINTER(GemmDesc), C.c_void_p, C.c_size_t, C.c_void_p]
        _lib.repq_pv.argtypes = [C.POINTER(PvDesc), C.c_void_p]
        _lib.repq_block_workspace_bytes.argtypes = [C.POINTER(BlockDesc), C.POINTER(C.c_size_t)]
        _lib.repq_block_forward.argtypes = [C.POINTER(BlockDesc), C.POINTER(BlockParams), C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_size_t, C.c_void_p]
        _lib.repq_device_status.argtypes = [C.POINTER(C.c_int32), C.c_int]
        _lib.repq_block_forward_timed.argtypes = [C.POINTER(BlockDesc), C.POINTER(BlockParams), C.c_void_p, C.c_void_p,
                                                  C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_float)]
        _lib.repq_block_forward_static.argtypes = [C.POINTER(BlockDesc), C.POINTER(BlockParams), C.c_void_p,
                                                   C.c_void_p, C.c_void_p]
        _lib.repq_attention.argtypes = [C.POINTER(AttentionDesc), C.c_void_p]
        _lib.repq_block_forward_host.argtypes = [C.POINTER(BlockDesc), C.POINTER(BlockParams), C.POINTER(C.c_void_p),
                                                 C.POINTER(C.c_void_p), C.c_int, C.POINTER(HostStaging), C.c_void_p]
        _lib.repq_launch_count.restype = C.c_uint64
        _lib.repq_launch_count.argtypes = []
        _lib.repq_scale_zero_from_bounds.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        _lib.repq_fold_ln.argtypes = [C.c_int, C.c_int] + [C.c_void_p] * 12
        _lib.repq_pack_weights.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int64,
                                           C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.repq_rope_table.argtypes = [C.c_int, C.c_int, C.c_double, C.c_void_p]
        _lib.repq_layernorm.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int64, C.c_void_p, C.c_void_p, C.c_float,
                                        C.c_int, C.c_void_p, C.c_int64, C.c_void_p]
        _lib.repq_dual_clip.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_float,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.repq_bounded_wait_selftest.argtypes = [C.c_int64, C.c_void_p]
    return _lib


def repq_last_error() -> str:
    buf = C.create_string_buffer(1024)
    lib().repq_last_error(buf, 1024)
    return buf.value.decode("utf-8", "replace")


def _check(status: int) -> None:
    if status != REPQ_OK:
        raise RepqError(status, repq_last_error())


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    raise TypeError(type(t))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return REPQ_F32
    if t.dtype == torch.bfloat16:
        return REPQ_BF16
    raise TypeError("expected a float32 or bfloat16 tensor, got %s" % t.dtype)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def code_row_bytes(n: int, bits: int, align: int = 16) -> int:
    # bits may carry REPQ_BYTE_CODES (one byte per code) or be 6 | REPQ_PACKED6 (four codes in three bytes)
    raw = (n + 1) // 2 if bits == 4 else (n * 3 + 3) // 4 if bits == (6 | REPQ_PACKED6) else n
    return (raw + align - 1) // align * align


# ---------------------------------------------------------------------------------- host preparation

def repq_scale_zero_from_bounds(x_low, x_up, bits: int):
    lo = np.ascontiguousarray(np.atleast_1d(x_low), dtype=np.float32)
    hi = np.ascontiguousarray(np.atleast_1d(x_up), dtype=np.float32)
    s = np.empty_like(lo)
    z = np.empty(lo.shape, dtype=np.int32)
    _check(lib().repq_scale_zero_from_bounds(lo.size, _ptr(lo), _ptr(hi), bits, _ptr(s), _ptr(z)))
    return s, z


def repq_fold_ln(gamma, beta, s, z, W, b):
    gamma = np.ascontiguousarray(gamma, dtype=np.float32)
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    s = np.ascontiguousarray(s, dtype=np.float32)
    z = np.ascontiguousarray(z, dtype=np.int32)
    W = np.ascontiguousarray(W, dtype=np.float32)
    b = None if b is None else np.ascontiguousarray(b, dtype=np.float32)
    N, D = W.shape
    gamma_t, beta_t = np.empty_like(gamma), np.empty_like(beta)
    W_t, b_t = np.empty_like(W), np.empty(N, dtype=np.float32)
    s_t, z_t = C.c_float(), C.c_int32()
    _check(lib().repq_fold_ln(D, N, _ptr(gamma), _ptr(beta), _ptr(s), _ptr(z), _ptr(W), _ptr(b), _ptr(gamma_t),
                              _ptr(beta_t), C.addressof(s_t), C.addressof(z_t), _ptr(W_t), _ptr(b_t)))
    return gamma_t, beta_t, float(s_t.value), int(z_t.value), W_t, b_t


def repq_pack_weights(W, bits_w: int):
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    ld = code_row_bytes(K, bits_w)
    codes = np.empty((N, ld), dtype=np.uint8)
    s_w = np.empty(N, dtype=np.float32)
    z_w = np.empty(N, dtype=np.int32)
    wsum = np.empty(N, dtype=np.int32)
    _check(lib().repq_pack_weights(N, K, bits_w, _ptr(W), _ptr(codes), ld, _ptr(s_w), _ptr(z_w), _ptr(wsum)))
    return codes, s_w, z_w, wsum


# ---------------------------------------------------------------------------------- device stages

def repq_ln_quant(x: torch.Tensor, gamma_t: torch.Tensor, beta_t: torch.Tensor, eps: float, s_t: float, z_t: int,
                  bits: int, codes: torch.Tensor, row_sum: Optional[torch.Tensor] = None,
                  norm_kind: int = REPQ_NORM_LAYERNORM, stream=None) -> None:
    rows, D = x.shape
    _check(lib().repq_ln_quant(_ptr(x), _dtype_code(x), rows, D, x.stride(0), _ptr(gamma_t), _ptr(beta_t), eps,
                               norm_kind, s_t, z_t, bits, _ptr(codes), codes.stride(0), _ptr(row_sum),
                               _stream(stream)))


def repq_softmax_log2(scores: torch.Tensor, L: int, s: float, bits: int, codes: torch.Tensor,
                      pre_scale: float = 1.0, causal_period: int = 0, causal_offset: int = 0, stream=None) -> None:
    rows = scores.shape[0]
    _check(lib().repq_softmax_log2(_ptr(scores), _dtype_code(scores), rows, L, scores.stride(0), pre_scale,
                                   causal_period, causal_offset, s, bits, _ptr(codes), codes.stride(0),
                                   _stream(stream)))


def repq_qgemm_workspace_bytes(d: GemmDesc) -> int:
    n = C.c_size_t()
    _check(lib().repq_qgemm_workspace_bytes(C.byref(d), C.byref(n)))
    return int(n.value)


def repq_qgemm(d: GemmDesc, workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().repq_qgemm(C.byref(d), _ptr(workspace), nbytes, _stream(stream)))


def repq_pv(d: PvDesc, stream=None) -> None:
    _check(lib().repq_pv(C.byref(d), _stream(stream)))


def repq_attention(d: AttentionDesc, stream: Optional[int] = None) -> None:
    _check(lib().repq_attention(C.byref(d), _stream(stream)))


def repq_block_workspace_bytes(d: BlockDesc) -> int:
    n = C.c_size_t()
    _check(lib().repq_block_workspace_bytes(C.byref(d), C.byref(n)))
    return int(n.value)


def repq_block_forward(d: BlockDesc, p: BlockParams, x: torch.Tensor, y: torch.Tensor, workspace: torch.Tensor,
                       stream=None) -> None:
    nbytes = workspace.numel() * workspace.element_size()
    _check(lib().repq_block_forward(C.byref(d), C.byref(p), _ptr(x), _ptr(y), _ptr(workspace), nbytes,
                                    _stream(stream)))


def repq_block_forward_timed(d: BlockDesc, p: BlockParams, x: torch.Tensor, y: torch.Tensor, workspace: torch.Tensor,
                             stream=None):
    """Like repq_block_forward, but synchronises and returns the per-stage durations in milliseconds."""
    nbytes = workspace.numel() * workspace.element_size()
    ms = (C.c_float * REPQ_BLOCK_STAGES)()
    _check(lib().repq_block_forward_timed(C.byref(d), C.byref(p), _ptr(x), _ptr(y), _ptr(workspace), nbytes,
                                          _stream(stream), ms))
    return [float(v) for v in ms]


def repq_block_forward_static(d: BlockDesc, p: BlockParams, x: torch.Tensor, y: torch.Tensor, stream=None) -> None:
    """repq_block_forward without a workspace argument: the library's built-in 8 MiB scratch array is used,
    so nothing is allocated.  For hosts that may not allocate device memory on the inference path; blocks that
    need more scratch are rejected.  Calls share the scratch: do not overlap them on one GPU."""
    _check(lib().repq_block_forward_static(C.byref(d), C.byref(p), _ptr(x), _ptr(y), _stream(stream)))


class HostStaging(C.Structure):
    _fields_ = [("x_dev", C.c_void_p * 2), ("y_dev", C.c_void_p * 2), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t)]


def repq_block_forward_host(d: BlockDesc, p: BlockParams, x_host, y_host, x_dev, y_dev, workspace: torch.Tensor,
                            stream=None) -> None:
    """Block over a sequence of batches held in host memory: x_host / y_host are lists of (pinned) CPU tensors,
    x_dev / y_dev pairs of device staging tensors.  Copies and kernels of neighbouring batches overlap; the
    results are valid once `stream` has completed."""
    n = len(x_host)
    assert len(y_host) == n and len(x_dev) == 2 and len(y_dev) == 2
    xs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in x_host])
    ys = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in y_host])
    st = HostStaging()
    for k in range(2):
        st.x_dev[k] = _ptr(x_dev[k])
        st.y_dev[k] = _ptr(y_dev[k])
    st.workspace = _ptr(workspace)
    st.workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().repq_block_forward_host(C.byref(d), C.byref(p), xs, ys, n, C.byref(st), _stream(stream)))


def repq_launch_count() -> int:
    return int(lib().repq_launch_count())


def repq_device_status(reset: bool = False) -> int:
    """The device's health word (0 = healthy).  REPQ_TIMEOUT from the library is the non-zero word, not an error
    of this call."""
    v = C.c_int32()
    st = lib().repq_device_status(C.byref(v), int(reset))
    if st != REPQ_TIMEOUT:
        _check(st)
    return int(v.value)


def repq_bounded_wait_selftest(limit_cycles: int, stream=None) -> None:
    _check(lib().repq_bounded_wait_selftest(int(limit_cycles), _stream(stream)))


def repq_layernorm(x: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor, eps: float, y: torch.Tensor,
                   norm_kind: int = REPQ_NORM_LAYERNORM, stream=None) -> None:
    """Full-precision normalisation of a calibration batch (float32 out), the input of repq_dual_clip."""
    rows, D = x.shape
    _check(lib().repq_layernorm(_ptr(x), _dtype_code(x), rows, D, x.stride(0), _ptr(gamma), _ptr(beta), eps, norm_kind,
                                _ptr(y), y.stride(0), _stream(stream)))


def repq_dual_clip(x: torch.Tensor, bits: int, x_low: torch.Tensor, x_up: torch.Tensor, loss: Optional[torch.Tensor] = None,
                   iters: int = 100, lr: float = 0.01, alpha0: float = 0.0, stream=None) -> None:
    """Per-channel dual clipping on device activations x [n, D] float32: learned bounds into x_low / x_up [D]."""
    n, D = x.shape
    _check(lib().repq_dual_clip(_ptr(x), n, D, x.stride(0), bits, iters, lr, alpha0, _ptr(x_low), _ptr(x_up), _ptr(loss),
                                _stream(stream)))


def repq_rope_table(seq: int, d_h: int, base: float = 10000.0) -> np.ndarray:
    """(cos, sin) table of the rotary embedding, float32 [seq, d_h / 2, 2]."""
    t = np.empty((seq, d_h // 2, 2), dtype=np.float32)
    _check(lib().repq_rope_table(seq, d_h, float(base), _ptr(t)))
    return t


# ---------------------------------------------------------------------------------- descriptor helpers

def gemm_desc(M: int, N: int, K: int, a_codes: torch.Tensor, bits_a: int, s_a: float, z_a: int,
              w_codes: torch.Tensor, bits_w: int, out: torch.Tensor, *, s_w=None, z_w=None, s_w_scalar=1.0,
              z_w_scalar=0, a_row_sum=None, w_row_sum=None, bias=None, alpha=1.0, gelu=False, residual=None,
              out_kind=REPQ_OUT_F32, out_bits=8, out_scale: Sequence[float] = (1.0,), out_zero: Sequence[int] = (0,),
              out_row_sum=None, acc_debug=None, batch=(1, 1), a_strides=(0, 0), w_strides=(0, 0), o_strides=(0, 0),
              lda_bytes=None, ldw_bytes=None, ldo=None, causal=False, rope=None, rope_period=0, rope_dim=0,
              rope_groups=0, glu=False) -> GemmDesc:
    """Fills a GemmDesc from torch tensors (pointer and stride marshalling only)."""
    d = GemmDesc()
    d.M, d.N, d.K = M, N, K
    d.batch_outer, d.batch_inner = batch
    d.a_codes, d.bits_a = _ptr(a_codes), bits_a
    d.lda_bytes = a_codes.stride(0) if lda_bytes is None else lda_bytes
    d.a_stride_outer, d.a_stride_inner = a_strides
    d.s_a, d.z_a, d.a_row_sum = s_a, z_a, _ptr(a_row_sum)
    d.w_codes, d.bits_w = _ptr(w_codes), bits_w
    d.ldw_bytes = w_codes.stride(0) if ldw_bytes is None else ldw_bytes
    d.w_stride_outer, d.w_stride_inner = w_strides
    d.s_w, d.z_w, d.s_w_scalar, d.z_w_scalar = _ptr(s_w), _ptr(z_w), s_w_scalar, z_w_scalar
    d.w_row_sum, d.bias, d.alpha = _ptr(w_row_sum), _ptr(bias), alpha
    d.gelu = int(gelu)
    d.residual = _ptr(residual)
    d.residual_dtype = _dtype_code(residual) if residual is not None else 0
    d.ld_residual = residual.stride(0) if residual is not None else 0
    d.out_kind, d.out_bits, d.out_groups = out_kind, out_bits, len(out_scale)
    for i, (s, z) in enumerate(zip(out_scale, out_zero)):
        d.out_scale[i], d.out_zero[i] = s, z
    d.out = _ptr(out)
    d.ldo = out.stride(0) if ldo is None else ldo
    d.o_stride_outer, d.o_stride_inner = o_strides
    d.out_row_sum, d.acc_debug = _ptr(out_row_sum), _ptr(acc_debug)
    d.causal = int(causal)
    d.rope_cos_sin, d.rope_period, d.rope_dim, d.rope_groups = _ptr(rope), rope_period, rope_dim, rope_groups
    d.glu = int(glu)
    return d
