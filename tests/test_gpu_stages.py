"""Stage-level parity of the CUDA kernels against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest

from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2402_05628_b200.build import build_library
    build_library()


@pytest.mark.parametrize("rows,D,bits,bf16", [
    (197, 384, 4, False), (1000, 768, 4, True), (515, 768, 6, True), (333, 1024, 4, True),
    (130, 4096, 4, True), (67, 8192, 8, True), (9, 16384, 4, False), (1, 8, 4, False), (77, 200, 8, True),
    (4099, 768, 4, False), (5003, 1024, 4 | parity.BYTE_CODES, True), (2500, 2048, 6, True), (3001, 4096, 8, True),
    (1201, 8192, 4, True), (333, 1024, 4, False),
    # rows that do not fill their thread group: factors in registers (3200, 4088), factors in shared memory (1000, 1096)
    (257, 3200, 4, True), (99, 4088, 8, True), (301, 1000, 4, True), (150, 1096, 6, True),
])
def test_ln_quant_matches_channelwise_oracle(rows, D, bits, bf16):
    rep = parity.check_ln_quant(rows, D, bits, bf16, seed=rows + D)
    assert rep["bad"] == 0, rep
    assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep


@pytest.mark.parametrize("D", [4096, 8192, 768, 1024, 2048])
def test_ln_quant_mean_free_without_row_sums_repeated(D):
    """Mean-free normalisation without row sums runs one reduction per row (one barrier per iteration of a thread
    group wider than a warp): repeated launches over many rows per block agree with the oracle and one another."""
    rep = parity.check_ln_quant(20000, D, 4, True, seed=D, rms=True, eps=1e-5, want_sum=False, runs=6)
    assert rep["bad"] == 0, rep
    assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep


def test_ln_quant_rms_strided_and_empty():
    assert parity.check_ln_quant(300, 4096, 4, True, seed=3, rms=True, eps=1e-5)["bad"] == 0
    assert parity.check_ln_quant(300, 768, 4, True, seed=4, pad_cols=8)["bad"] == 0
    assert parity.check_ln_quant(300, 768, 8, False, seed=5, want_sum=False)["bad"] == 0
    assert parity.check_ln_quant(0, 768, 4, True, seed=6)["total"] == 0


@pytest.mark.parametrize("rows,L,bits,bf16", [
    (1182, 197, 4, False), (700, 577, 4, False), (300, 2048, 8, False), (40, 8192, 4, False),
    (64, 197, 6, True), (5, 1, 4, False), (33, 7, 8, False), (20, 16384, 4, True),
])
def test_softmax_log2_matches_logsqrt2_oracle(rows, L, bits, bf16):
    rep = parity.check_softmax_log2(rows, L, bits, bf16, seed=rows + L)
    assert rep["bad"] == 0, rep
    assert rep["mismatch"] <= max(2, 2e-4 * rep["total"]), rep


def test_softmax_log2_variants():
    assert parity.check_softmax_log2(512, 256, 8, seed=1, causal_period=256)["bad"] == 0
    assert parity.check_softmax_log2(394, 197, 4, seed=2, causal_period=197)["bad"] == 0
    assert parity.check_softmax_log2(300, 197, 4, seed=3, s=0.7)["bad"] == 0
    assert parity.check_softmax_log2(300, 197, 4, seed=4, pre_scale=0.125)["bad"] == 0
    assert parity.check_softmax_log2(300, 197, 4, seed=5, ld_pad=197)["bad"] == 0      # unaligned rows
    assert parity.check_softmax_log2(300, 197, 8, seed=6, ld_pad=208)["bad"] == 0      # stride beyond the last chunk
    assert parity.check_softmax_log2(70, 577, 6, seed=7, ld_pad=584)["bad"] == 0       # whole last chunk in the stride
    assert parity.check_softmax_log2(70, 581, 4, seed=8, ld_pad=584)["bad"] == 0       # stride ends inside the last chunk


@pytest.mark.parametrize("M,N,K,ba,bw", [
    (64, 64, 64, 8, 8), (197, 1152, 384, 4, 4), (130, 72, 100, 4, 4), (33, 17, 50, 8, 8), (257, 200, 333, 6, 6),
    (1, 8, 16, 4, 8), (300, 96, 11008, 4, 4), (64, 64, 4000, 8, 8),
])
def test_qgemm_accumulators_and_float_output(M, N, K, ba, bw):
    parity.check_qgemm(M, N, K, ba, bw, seed=M + N + K)


def test_qgemm_epilogues():
    parity.check_qgemm(300, 192, 256, 4, 4, out_kind="bf16", seed=1)
    parity.check_qgemm(300, 192, 256, 4, 4, out_kind="f32", residual="bf16", seed=2)
    parity.check_qgemm(300, 192, 256, 4, 4, out_kind="bf16", residual="f32", gelu=True, seed=3)
    parity.check_qgemm(300, 192, 256, 4, 4, out_kind="codes", groups=3, out_bits=4, seed=4)
    parity.check_qgemm(300, 192, 256, 8, 8, out_kind="codes", gelu=True, out_bits=8, want_out_sum=True, seed=5)
    parity.check_qgemm(300, 192, 256, 6, 6, out_kind="codes", out_bits=6, want_out_sum=True, give_sums=True, seed=6)


@pytest.mark.parametrize("Bn,H,Lq,Lk,dh,bp,bv,causal", [
    (2, 3, 197, 197, 64, 4, 4, False), (1, 2, 577, 577, 64, 4, 4, False), (1, 2, 300, 300, 128, 8, 4, True),
    (2, 2, 64, 64, 32, 6, 6, False), (1, 1, 1, 130, 16, 8, 8, False), (1, 2, 100, 260, 64, 4, 8, True),
    (1, 1, 70, 70, 96, 8, 8, True),
])
def test_pv_matches_oracle(Bn, H, Lq, Lk, dh, bp, bv, causal):
    parity.check_pv(Bn, H, Lq, Lk, dh, bp, bv, causal, seed=Lq + dh)


def test_pv_epilogues():
    parity.check_pv(2, 2, 197, 197, 64, 4, 4, out_kind="bf16", seed=1)
    parity.check_pv(2, 2, 197, 197, 64, 4, 4, out_kind="codes", out_bits=4, want_out_sum=True, seed=2)
    parity.check_pv(1, 2, 130, 130, 128, 8, 4, causal=True, out_kind="codes", out_bits=8, want_out_sum=True, seed=3, s_p=0.7)


@pytest.mark.parametrize("Bn,H,Lq,Lk,dh,bits,causal", [
    (2, 3, 197, 197, 64, 4, False), (1, 2, 577, 577, 64, 4, False), (1, 2, 300, 300, 128, 4, True),
    (2, 2, 70, 70, 32, 8, False), (1, 1, 1, 130, 16, 6, False), (1, 2, 100, 260, 48, 4, True),
    (1, 2, 50, 50, 24, 4, False),      # head size not a multiple of 16: generic warp-MMA kernel
])
def test_scores_match_oracle(Bn, H, Lq, Lk, dh, bits, causal):
    parity.check_scores(Bn, H, Lq, Lk, dh, bits, causal, seed=Lq + dh)


def test_four_bit_quantizers_stored_one_code_per_byte():
    """REPQ_BYTE_CODES changes the storage of the codes, not the quantizer: same oracle, byte-wide containers."""
    b4 = 4 | parity.BYTE_CODES
    assert parity.check_ln_quant(515, 768, b4, True, seed=11)["bad"] == 0
    assert parity.check_softmax_log2(300, 197, b4, seed=12)["bad"] == 0
    parity.check_qgemm(300, 192, 256, b4, b4, out_kind="codes", groups=3, out_bits=b4, seed=13)
    parity.check_qgemm(197, 1152, 384, b4, 4, out_kind="codes", out_bits=b4, want_out_sum=True, gelu=True, seed=14)
    parity.check_qgemm(130, 72, 100, 4, b4, seed=15)
    parity.check_pv(2, 2, 197, 197, 64, 4, b4, out_kind="codes", out_bits=b4, want_out_sum=True, seed=16)
    parity.check_pv(1, 2, 130, 130, 128, b4, b4, causal=True, seed=17)
    parity.check_scores(2, 3, 197, 197, 64, b4, seed=18)
    parity.check_scores(1, 2, 50, 50, 24, b4, seed=19)


@pytest.mark.parametrize("Bn,H,L,dh,bp,bv", [(3, 12, 256, 64, 4, 4 | parity.BYTE_CODES), (1, 4, 600, 128, 8, 4), (2, 3, 197, 32, 6, 6)])
def test_pv_repeated_launches_reproduce_the_oracle(Bn, H, L, dh, bp, bv):
    parity.check_pv_uniform_codes(Bn, H, L, dh, bp, bv, runs=12, seed=L)


@pytest.mark.parametrize("Bn,H,Lq,Lk,dh,bits,causal", [
    (2, 3, 197, 197, 64, 4 | parity.BYTE_CODES, False), (1, 2, 577, 577, 64, 4 | parity.BYTE_CODES, False),
    (1, 2, 300, 300, 128, 4 | parity.BYTE_CODES, True), (1, 2, 100, 260, 48, 8, True), (1, 1, 513, 513, 16, 6, False),
    (1, 3, 130, 700, 96, 4 | parity.BYTE_CODES, True),
])
def test_scores_from_byte_codes_match_oracle(Bn, H, Lq, Lk, dh, bits, causal):
    parity.check_scores(Bn, H, Lq, Lk, dh, bits, causal, seed=Lq + dh + 1)


@pytest.mark.parametrize("Bn,H,Lq,Lk,dh,bits,bp,causal", [
    (2, 3, 197, 197, 64, 4, 4, False), (1, 2, 577, 577, 64, 4, 4, False), (1, 2, 300, 300, 128, 4, 8, True),
    (2, 2, 64, 64, 32, 6, 6, False), (1, 1, 1, 130, 16, 8, 8, False), (1, 2, 100, 260, 48, 4, 4, True),
    (1, 1, 70, 70, 96, 8, 4, True), (1, 2, 700, 700, 64, 4, 4, True), (1, 2, 150, 150, 128, 6, 6, False),
    (1, 2, 300, 300, 64, 4, 6, True),
    # wide heads (visits of 128 keys, two issuing warps): one visit, a visit with a single key, odd and even numbers of
    # visits, every score form and code width, head sizes that do not fill the tile, keys beyond the queries under a mask
    (1, 2, 128, 128, 128, 4, 8, False), (1, 1, 129, 129, 128, 4, 4, True), (1, 2, 260, 1000, 128, 4, 8, True),
    (1, 1, 200, 700, 128, 8, 8, False), (1, 2, 140, 385, 80, 4, 6, False), (1, 1, 257, 640, 112, 6, 8, True),
    (2, 1, 33, 1030, 96, 4, 4, True),
])
def test_fused_attention_matches_oracle(Bn, H, Lq, Lk, dh, bits, bp, causal):
    parity.check_attention(Bn, H, Lq, Lk, dh, bits, bp, causal, seed=Lq + dh)


def test_fused_attention_epilogues():
    parity.check_attention(2, 2, 197, 197, 64, 4, 4, out_kind="bf16", seed=1)
    parity.check_attention(2, 2, 197, 197, 64, 4, 4, out_kind="codes", out_bits=4 | parity.BYTE_CODES, seed=2)
    parity.check_attention(1, 2, 130, 130, 128, 4, 8, causal=True, out_kind="codes", out_bits=8, seed=3, s_p=0.7)
    parity.check_attention(1, 2, 130, 130, 64, 4, 4, out_kind="codes", out_bits=4, seed=4)


@pytest.mark.parametrize("M,N,K,bits,out_bits,groups,gelu,residual,out_kind", [
    # byte codes of 4 and 6 bits through the comparison-free quantizer: one and three column groups (group edges on
    # and off the 64-column slices), GELU in front of it, rows that end inside a tile
    (700, 768, 256, 4, 4, 1, False, None, "codes"), (700, 768, 256, 4, 4, 3, False, None, "codes"),
    (389, 576, 384, 4, 4, 3, False, None, "codes"), (700, 512, 256, 6, 6, 1, True, None, "codes"),
    (260, 1024, 128, 4, 6, 1, True, None, "codes"),
    # 8-bit byte codes and packed 4-bit codes keep the clamping quantizer
    (700, 512, 256, 8, 8, 2, False, None, "codes"), (300, 256, 256, 4, -4, 1, False, None, "codes"),
    # float outputs with both residual types, ragged last column tile
    (700, 768, 256, 4, 4, 1, False, "bf16", "bf16"), (389, 448, 768, 6, 4, 1, False, "f32", "f32"),
    (513, 200, 256, 4, 4, 1, True, "bf16", "bf16"),
])
def test_qgemm_common_epilogue_path(M, N, K, bits, out_bits, groups, gelu, residual, out_kind):
    """The epilogue the block runs (no accumulator dump, so the per-warp column terms, the bulk stores and the
    comparison-free quantizer are what is checked), output against the oracle."""
    b = bits | parity.BYTE_CODES
    ob = -out_bits if out_bits < 0 else (out_bits | parity.BYTE_CODES)              # negative: packed 4-bit output
    parity.check_qgemm(M, N, K, b, b, out_kind=out_kind, gelu=gelu, residual=residual, groups=groups, out_bits=ob,
                       want_acc=False, want_out_sum=(out_kind == "codes"), seed=M + N + K + groups)


@pytest.mark.parametrize("M,N,K,bits,out_kind", [
    (300, 768, 256, 4, "codes"), (400, 1536, 384, 4, "codes"), (150, 192, 128, 8, "codes"), (300, 768, 256, 4, "f32"),
    (50, 96, 64, 4, "codes"),                 # small: the warp-MMA kernel
])
def test_qgemm_rotary_embedding_in_the_epilogue(M, N, K, bits, out_kind):
    dh = 32 if N % 96 == 0 else 64
    parity.check_qgemm_pair_step(M, N, K, bits | parity.BYTE_CODES, "rope", out_kind=out_kind, seed=M + N, L=50, dh=dh)


@pytest.mark.parametrize("M,N,K,bits,out_kind", [
    (300, 1024, 256, 4, "codes"), (389, 2816, 512, 4, "codes"), (260, 640, 128, 8, "codes"), (300, 512, 256, 6, "f32"),
    (40, 96, 64, 4, "codes"),
])
def test_qgemm_gated_product_in_the_epilogue(M, N, K, bits, out_kind):
    parity.check_qgemm_pair_step(M, N, K, bits | parity.BYTE_CODES, "glu", out_kind=out_kind, seed=M + N)


@pytest.mark.parametrize("M,N,K,residual,out_kind", [
    (12608, 768, 768, "bf16", "bf16"),        # residual boxes by bulk tensor copies (short K)
    (4000, 768, 3072, "bf16", "bf16"),        # row-per-lane residual loads
    (3000, 512, 256, "f32", "f32"),
])
def test_qgemm_with_residual_repeated_launches(M, N, K, residual, out_kind):
    parity.check_qgemm_repeated(M, N, K, 4, residual, out_kind, runs=12, seed=K)


def test_bounded_wait_runs_out_and_the_context_survives():
    """A device-side wait that nothing ends returns after its limit, reports through the health word, and the
    next launches are correct."""
    import torch
    from paper_2402_05628_b200 import binding as B
    torch.cuda.synchronize()
    assert B.repq_device_status(reset=True) == 0
    B.repq_bounded_wait_selftest(2_000_000)               # about a millisecond of SM clock
    torch.cuda.synchronize()
    assert B.repq_device_status() == 77                    # the self-test's code; the library call says REPQ_TIMEOUT
    v = __import__("ctypes").c_int32()
    assert B.lib().repq_device_status(__import__("ctypes").byref(v), 1) == B.REPQ_TIMEOUT and v.value == 77
    assert B.repq_device_status() == 0                     # cleared by the reset above
    parity.check_qgemm(300, 192, 256, 4, 4, out_kind="bf16", seed=1)
    assert parity.check_ln_quant(300, 768, 4, True, seed=4)["bad"] == 0
    with pytest.raises(B.RepqError):
        B.repq_bounded_wait_selftest(0)


@pytest.mark.parametrize("n,D,bits,iters,strided", [
    (1500, 48, 4, 100, False), (6304, 384, 4, 100, False), (700, 100, 8, 30, True), (33, 7, 6, 10, False), (900, 64, 4, 0, False),
])
def test_dual_clip_matches_oracle(n, D, bits, iters, strided):
    rep = parity.check_dual_clip(n, D, bits, seed=n + D, iters=iters, strided=strided)
    if iters:
        assert rep["loss"] < rep["loss0"]


@pytest.mark.parametrize("rows,D,bits", [(262144, 768, 4), (65536, 4096, 4), (1048576, 384, 4 | parity.BYTE_CODES), (32768, 8192, 8)])
def test_ln_quant_at_sweep_sizes_sampled_rows(rows, D, bits):
    parity.check_ln_quant_sampled(rows, D, bits)


@pytest.mark.parametrize("rows,L,bits", [(151296, 197, 4), (151296, 577, 8), (32768, 2048, 4), (32768, 8192, 4)])
def test_softmax_log2_at_sweep_sizes_sampled_rows(rows, L, bits):
    parity.check_softmax_log2_sampled(rows, L, bits)


@pytest.mark.parametrize("M,N,K,qbits,out_kind,weights", [
    (16384, 2304, 768, 4, "codes", "bytes"), (16384, 768, 3072, 8, "bf16", "bytes"), (16384, 12288, 4096, 4, "codes", "bytes"),
    (16384, 4096, 11008, 4, "bf16", "bytes"), (65536, 768, 768, 4, "codes", "bytes"), (2048, 4096, 4096, 8, "codes", "bytes"),
    (16384, 11008, 4096, 4, "codes", "packed"), (8192, 4096, 11008, 4, "bf16", "packed"),
    (12608, 2304, 768, 6, "codes", "packed"), (8192, 4096, 4096, 6, "bf16", "packed"),
])
def test_qgemm_at_sweep_sizes_sampled_rows(M, N, K, qbits, out_kind, weights):
    parity.check_qgemm_sampled(M, N, K, qbits, out_kind, weights=weights)


def test_dual_clip_leaves_a_constant_channel_alone():
    import torch
    from paper_2402_05628_b200 import binding as B
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(3)
    x = torch.randn(500, 16, device=dev, generator=g)
    x[:, 5] = 0.75                      # a constant channel: Eq. 6 has no scale for it
    x[:, 9] = 0.0
    lo, hi = torch.empty(16, device=dev), torch.empty(16, device=dev)
    loss = torch.empty(32, dtype=torch.float64, device=dev)
    B.repq_dual_clip(x, 4, lo, hi, loss, iters=20, lr=0.01, alpha0=0.0)
    torch.cuda.synchronize()
    assert torch.isfinite(lo).all() and torch.isfinite(hi).all() and torch.isfinite(loss).all()
    assert float(lo[5]) == float(hi[5]) == 0.375 and float(lo[9]) == float(hi[9]) == 0.0       # sigmoid(0) = 1/2 of the extremes
    assert float(loss[5]) == 0.0 and float(loss[16 + 5]) == 0.0
    assert (hi[[0, 1, 2]] > lo[[0, 1, 2]]).all()


@pytest.mark.parametrize("M,N,K,out_kind", [
    (300, 192, 256, "f32"), (389, 576, 384, "codes"), (700, 512, 1000, "bf16"), (130, 72, 100, "f32"), (33, 17, 50, "f32"),
    (64, 64, 4, "f32"),
])
def test_qgemm_six_bit_weights_packed_four_to_three_bytes(M, N, K, out_kind):
    """Weights stored 6 | REPQ_PACKED6 (tensor-core kernel: expanded in shared memory; small or ragged shapes: the
    warp-MMA kernel), int32 accumulators bit-exact where they are dumped."""
    b6 = 6 | parity.BYTE_CODES
    parity.check_qgemm(M, N, K, b6, 6 | parity.PACKED6, out_kind=out_kind, out_bits=b6, seed=M + K, give_sums=(M % 2 == 0),
                       want_acc=(out_kind == "f32"))
