"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the header
declares, and its host entry points (Eq. 6, Eqs. 10-14 fold, weight packing) agree with the oracle."""
import os
import re

import numpy as np
import pytest

from oracle import repq_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2402_05628_b200.build import build_library
    build_library()
    from paper_2402_05628_b200 import binding
    binding.lib()
    return binding


def test_exports_match_header(B):
    header = open(os.path.join(ROOT, "include", "repq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(repq_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    lib = B.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), "library does not export %s" % name
    assert declared == set(B.EXPORTS)
    assert lib.repq_abi_version() == 5


def test_scale_zero_from_bounds_matches_oracle(B):
    rng = np.random.default_rng(0)
    lo = rng.normal(-1, 1, 500).astype(np.float32)
    hi = (lo + rng.uniform(0.1, 5, 500)).astype(np.float32)
    for bits in (4, 6, 8):
        s, z = B.repq_scale_zero_from_bounds(lo, hi, bits)
        s_ref, z_ref = orc.uniform_scale_zero(lo, hi, bits)
        assert np.array_equal(s.astype(np.float64), s_ref)
        assert np.array_equal(z.astype(np.int64), z_ref)
    with pytest.raises(B.RepqError) as e:
        B.repq_scale_zero_from_bounds(np.array([1.0]), np.array([0.5]), 4)
    assert e.value.status == B.REPQ_INVALID_ARG and "x_up" in str(e.value)
    with pytest.raises(B.RepqError):
        B.repq_scale_zero_from_bounds(lo, hi, 5)


def test_fold_ln_matches_oracle(B):
    rng = np.random.default_rng(1)
    D, N = 96, 40
    gamma = rng.normal(1, 0.1, D).astype(np.float32)
    beta = rng.normal(0, 0.1, D).astype(np.float32)
    s = rng.lognormal(-2, 1, D).astype(np.float32)
    z = rng.integers(-3, 19, D).astype(np.int32)
    W = rng.normal(0, 0.02, (N, D)).astype(np.float32)
    b = rng.normal(0, 0.02, N).astype(np.float32)
    g_t, b_t, s_t, z_t, W_t, bias_t = B.repq_fold_ln(gamma, beta, s, z, W, b)
    rp = orc.reparam_layernorm(gamma, beta, s, z, W, b)
    assert z_t == rp["z_t"]
    assert abs(s_t - rp["s_t"]) <= np.spacing(np.float32(rp["s_t"]))
    for got, ref in ((g_t, rp["gamma_t"]), (b_t, rp["beta_t"]), (W_t, rp["W_t"]), (bias_t, rp["b_t"])):
        tol = np.abs(ref) * 2.0 ** -23 + 1e-12
        assert np.all(np.abs(got.astype(np.float64) - ref) <= tol)
    # no-bias form and the trivial case
    _, _, _, _, _, bias0 = B.repq_fold_ln(gamma, beta, s, z, W, None)
    assert np.allclose(bias0, rp["b_t"] - b, atol=1e-6)
    g1, b1, s1, z1, W1, bb1 = B.repq_fold_ln(gamma, beta, np.full(D, 0.125, np.float32), np.full(D, 7, np.int32), W, b)
    assert s1 == 0.125 and z1 == 7 and np.array_equal(g1, gamma) and np.array_equal(W1, W) and np.array_equal(bb1, b)


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_pack_weights_matches_oracle(B, bits):
    from tests.parity import unpack_codes
    rng = np.random.default_rng(bits)
    N, K = 33, 72
    W = rng.normal(0, 0.02, (N, K)).astype(np.float32)
    W[4] = 0.0
    W[5] = np.abs(W[5])
    codes, s_w, z_w, wsum = B.repq_pack_weights(W, bits)
    q_ref, s_ref, z_ref = orc.quant_weight_rtn(W, bits)
    assert codes.shape[1] % 16 == 0
    q = unpack_codes(codes, K, bits)
    assert np.array_equal(q, q_ref)
    assert np.array_equal(s_w.astype(np.float64), s_ref) and np.array_equal(z_w.astype(np.int64), z_ref)
    assert np.array_equal(wsum.astype(np.int64), q_ref.sum(axis=1))


def test_device_entry_points_validate_arguments_without_gpu(B):
    """Argument errors are reported before any CUDA call."""
    lib = B.lib()
    assert lib.repq_ln_quant(None, 0, 4, 64, 64, None, None, 1e-6, 0, 1.0, 0, 4, None, 32, None, None) == B.REPQ_INVALID_ARG
    assert "NULL" in B.repq_last_error()
    assert lib.repq_ln_quant(None, 0, 0, 64, 64, None, None, 1e-6, 0, 1.0, 0, 4, None, 32, None, None) == B.REPQ_OK
    assert lib.repq_softmax_log2(None, 0, 4, 64, 64, 1.0, 0, 0, 1.0, 4, None, 32, None) == B.REPQ_INVALID_ARG
    assert lib.repq_softmax_log2(16, 0, 4, 64, 64, 1.0, 0, 0, -1.0, 4, 16, 32, None) == B.REPQ_INVALID_ARG
    assert lib.repq_softmax_log2(16, 0, 4, 64, 64, 1.0, 0, 0, 1.0, 5, 16, 32, None) == B.REPQ_INVALID_ARG
    assert lib.repq_ln_quant(16, 0, 4, 60, 64, 16, 16, 1e-6, 0, 1.0, 0, 4, 16, 32, None, None) == B.REPQ_UNSUPPORTED
    assert lib.repq_ln_quant(16, 0, 4, 64, 64, 16, 16, 1e-6, 0, 1.0, 0, 4, 18, 32, None, None) == B.REPQ_ALIGNMENT


def test_rope_table_rotates_like_the_oracle(B):
    """The library's (cos, sin) table applied to a matrix gives the oracle's rotary embedding (float32 table against
    float64 angles: a few units of 2^-24 per entry)."""
    rng = np.random.default_rng(9)
    L, H, dh = 37, 2, 32
    t = B.repq_rope_table(L, dh, 10000.0).astype(np.float64)          # [L, dh/2, 2]
    X = rng.normal(size=(2 * L, H * dh))
    ref = orc.rope(X, 2, L, H, 10000.0)
    cos = np.tile(t[:, :, 0], (2, H))
    sin = np.tile(t[:, :, 1], (2, H))
    got = np.empty_like(X)
    got[:, 0::2] = X[:, 0::2] * cos - X[:, 1::2] * sin
    got[:, 1::2] = X[:, 0::2] * sin + X[:, 1::2] * cos
    assert np.abs(got - ref).max() < 4e-7 * np.abs(X).max()
    assert t[0, :, 0].tolist() == [1.0] * (dh // 2) and t[0, :, 1].tolist() == [0.0] * (dh // 2)
    with pytest.raises(B.RepqError):
        B.repq_rope_table(L, 7, 10000.0)


def test_pack_weights_six_bit_layout(B):
    """6 | REPQ_PACKED6: the same codes as the byte form, four to three bytes, code i in bits [6i, 6i + 6)."""
    from tests.parity import PACKED6, BYTE_CODES, pack_codes
    rng = np.random.default_rng(12)
    W = rng.normal(0, 0.02, (9, 53)).astype(np.float32)
    c8, s8, z8, sum8 = B.repq_pack_weights(W, 6 | BYTE_CODES)
    c6, s6, z6, sum6 = B.repq_pack_weights(W, 6 | PACKED6)
    assert np.array_equal(s8, s6) and np.array_equal(z8, z6) and np.array_equal(sum8, sum6)
    assert c6.shape[1] == B.code_row_bytes(53, 6 | PACKED6) == 48
    assert np.array_equal(c6, pack_codes(c8[:, :53], 6 | PACKED6, c6.shape[1]))
    bits = np.unpackbits(c6, axis=1, bitorder="little")[:, : 53 * 6].reshape(9, 53, 6)
    assert np.array_equal((bits * (1 << np.arange(6))).sum(axis=2), c8[:, :53])
