// Internal launchers shared between translation units of the repq library.
#pragma once
#include "common.h"
#include "epilogue.cuh"

namespace repq {

// Row sums of a code matrix: out[r] = sum_c codes[r, c] (zero-point correction terms).
repq_status launch_row_sum(const uint8_t* codes, int bits, int64_t rows, int64_t n, int64_t ld_bytes,
                           int32_t* out, cudaStream_t st);

// 4-bit packed codes -> one code per byte (dst rows of ld_dst bytes, zero-padded up to n_pad codes).
repq_status launch_expand4(const uint8_t* src, int64_t rows, int64_t n, int64_t ld_src, uint8_t* dst,
                           int64_t ld_dst, int64_t n_pad, cudaStream_t st);

// Warp-MMA integer GEMM (any shape, batched).
repq_status qgemm_mma(const repq_gemm_desc& d, const EpilogueParams& ep, cudaStream_t st);

// Attention-score kernel: batched code-by-code products with scalar quantizers, K <= 128, float32 output.
bool scores_supported(const repq_gemm_desc& d);
repq_status launch_scores(const repq_gemm_desc& d, cudaStream_t st);
// The same on tcgen05 (byte codes, 16-byte aligned operand rows and output rows); call only if scores_supported.
bool scores_tc_supported(const repq_gemm_desc& d);
repq_status launch_scores_tc(const repq_gemm_desc& d, cudaStream_t st);

// Tensor-memory (tcgen05) integer GEMM: plain (unbatched) products with TMA-compatible operands.
bool qgemm_tc_supported(const repq_gemm_desc& d);
size_t qgemm_tc_workspace(const repq_gemm_desc& d);
repq_status qgemm_tc(const repq_gemm_desc& d, const EpilogueParams& ep, void* ws, size_t ws_bytes,
                     cudaStream_t st);

// P.V (Eqs. 16-17): kernel parameters shared by the two implementations, storage widths already resolved
// (bits_v is 4 for packed codes, 8 for byte codes).
struct PvParams {
  const uint8_t* p; int bits_p; int64_t ldp, p_pair;
  const uint8_t* v; int bits_v; int64_t ldv, v_so, v_si;
  int Lq, Lk, d_h, batch_inner, causal;
  int z_v;
  float scale;               // s_p * s_v
  int out_kind, qmax, pack4;
  float inv_so; int zo;
  void* out; int64_t ldo, o_so, o_si;
  int32_t* out_row_sum;
};
// Tensor-memory (tcgen05) P.V kernel: needs V rows that allow vector loads; the warp-MMA kernel covers the rest.
bool pv_tc_supported(const repq_pv_desc& d);
repq_status launch_pv_tc(const repq_pv_desc& d, const PvParams& P, cudaStream_t st);

// One-thread kernel whose mbarrier wait can only run out (see repq_bounded_wait_selftest).
repq_status launch_wait_selftest(long long limit_cycles, cudaStream_t st);

// Device-side health word (bounded waits report here instead of trapping); nullptr on failure.
int32_t* device_status_word();

}  // namespace repq
