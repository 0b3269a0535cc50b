// repq_qgemm: argument validation, path selection and the small helper kernels (row sums, 4-bit
// expansion) around the two integer-GEMM kernels.
#include "kernels.h"

namespace repq {
namespace {

__global__ void row_sum_kernel(const uint8_t* __restrict__ codes, int bits, int64_t rows, int64_t n,
                               int64_t ld, int32_t* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = (int64_t(gridDim.x) * blockDim.x) >> 5;
  const int64_t nbytes = bits == 4 ? (n >> 1) : n;
  for (int64_t r = warp; r < rows; r += nwarps) {
    const uint8_t* p = codes + r * ld;
    int s = 0;
    if (bits == 6) {
      // four codes in three bytes (padding bits of the last group are zero): byte-wise, 24 bits at a time
      const int64_t nb6 = (n * 3 + 3) / 4;
      for (int64_t g = lane; g * 3 < nb6; g += 32) {
        uint32_t f = p[3 * g];
        if (3 * g + 1 < nb6) f |= uint32_t(p[3 * g + 1]) << 8;
        if (3 * g + 2 < nb6) f |= uint32_t(p[3 * g + 2]) << 16;
        s += int((f & 0x3Fu) + ((f >> 6) & 0x3Fu) + ((f >> 12) & 0x3Fu) + (f >> 18));
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) out[r] = s;
      continue;
    }
    const bool vec = (reinterpret_cast<uintptr_t>(p) & 15) == 0;
    int64_t b = 0;
    if (vec) {
      for (b = int64_t(lane) * 16; b + 16 <= nbytes; b += 32 * 16) {
        const uint4 v = *reinterpret_cast<const uint4*>(p + b);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (bits == 4) {
            s = __dp4a(w[i] & 0x0F0F0F0Fu, 0x01010101u, uint32_t(s));
            s = __dp4a((w[i] >> 4) & 0x0F0F0F0Fu, 0x01010101u, uint32_t(s));
          } else {
            s = __dp4a(w[i], 0x01010101u, uint32_t(s));
          }
        }
      }
      b = nbytes / 16 * 16;
    }
    for (int64_t i = b + lane; i < nbytes; i += 32) s += bits == 4 ? (p[i] & 15) + (p[i] >> 4) : p[i];
    if (bits == 4 && (n & 1) && lane == 0) s += p[nbytes] & 15;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) out[r] = s;
  }
}

// Each thread expands 8 source bytes (16 codes) into 16 destination bytes.
__global__ void expand4_kernel(const uint8_t* __restrict__ src, int64_t rows, int64_t n, int64_t ld_src,
                               uint8_t* __restrict__ dst, int64_t ld_dst, int64_t n_pad) {
  const int64_t groups_per_row = n_pad / 16;
  const int64_t total = rows * groups_per_row;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += int64_t(gridDim.x) * blockDim.x) {
    const int64_t r = i / groups_per_row, gq = i % groups_per_row;
    const int64_t c0 = gq * 16;
    const uint8_t* s = src + r * ld_src + c0 / 2;
    uint32_t w[2] = {0u, 0u};
    if (c0 + 16 <= n && ((reinterpret_cast<uintptr_t>(s) & 7) == 0)) {
      const uint2 v = *reinterpret_cast<const uint2*>(s);
      w[0] = v.x; w[1] = v.y;
    } else {
      for (int e = 0; e < 8; ++e) {
        const int64_t c = c0 + 2 * e;
        uint32_t byte = 0;
        if (c < n) byte = s[e];
        if (c + 1 >= n) byte &= 0x0F;
        w[e >> 2] |= byte << (8 * (e & 3));
      }
    }
    uint4 o;
    uint32_t lo = w[0] & 0x0F0F0F0Fu, hi = (w[0] >> 4) & 0x0F0F0F0Fu;
    o.x = __byte_perm(lo, hi, 0x5140);
    o.y = __byte_perm(lo, hi, 0x7362);
    lo = w[1] & 0x0F0F0F0Fu; hi = (w[1] >> 4) & 0x0F0F0F0Fu;
    o.z = __byte_perm(lo, hi, 0x5140);
    o.w = __byte_perm(lo, hi, 0x7362);
    *reinterpret_cast<uint4*>(dst + r * ld_dst + c0) = o;
  }
}

repq_status validate(const repq_gemm_desc& d) {
  REPQ_REQUIRE(d.M >= 0 && d.N > 0 && d.K > 0, REPQ_INVALID_ARG, "qgemm: M >= 0, N > 0, K > 0 required");
  REPQ_REQUIRE(d.batch_outer > 0 && d.batch_inner > 0, REPQ_INVALID_ARG, "qgemm: batch counts must be positive");
  REPQ_REQUIRE(bits_ok(d.bits_a) && bits_w_ok(d.bits_w), REPQ_INVALID_ARG, "qgemm: bits must be 4, 6 or 8");
  if (d.M == 0) return REPQ_OK;
  REPQ_REQUIRE(d.a_codes && d.w_codes && d.out, REPQ_INVALID_ARG, "qgemm: NULL operand or output");
  REPQ_REQUIRE(d.lda_bytes >= code_row_bytes(d.K, d.bits_a) && d.ldw_bytes >= code_row_bytes(d.K, d.bits_w),
               REPQ_INVALID_ARG, "qgemm: operand row stride shorter than K codes");
  REPQ_REQUIRE(int64_t(d.K) * 255 * 255 < (int64_t(1) << 31), REPQ_UNSUPPORTED, "qgemm: K too large for int32 accumulators");
  REPQ_REQUIRE(d.s_a > 0.f, REPQ_INVALID_ARG, "qgemm: s_a must be positive");
  REPQ_REQUIRE(d.out_kind == REPQ_OUT_F32 || d.out_kind == REPQ_OUT_BF16 || d.out_kind == REPQ_OUT_CODES,
               REPQ_INVALID_ARG, "qgemm: unknown out_kind");
  const bool batched = d.batch_outer * int64_t(d.batch_inner) > 1;
  if (batched)
    REPQ_REQUIRE(!d.residual && !d.acc_debug && !d.out_row_sum && !d.a_row_sum && !d.w_row_sum, REPQ_UNSUPPORTED,
                 "qgemm: residual / row sums / acc_debug are for plain (unbatched) products");
  if (packed6(d.bits_w))
    REPQ_REQUIRE(!batched, REPQ_UNSUPPORTED, "qgemm: REPQ_PACKED6 is for the weights of a plain (unbatched) product");
  const int n_out = d.glu ? d.N / 2 : d.N;        // output columns
  if (d.glu) {
    REPQ_REQUIRE(d.out_groups <= 1, REPQ_UNSUPPORTED, "qgemm: glu takes one output group");
    REPQ_REQUIRE(!(d.out_kind == REPQ_OUT_CODES && packed4(d.out_bits)), REPQ_UNSUPPORTED,
                 "qgemm: glu writes float outputs or codes stored one per byte");
  }
  if (d.out_kind == REPQ_OUT_CODES) {
    REPQ_REQUIRE(bits_ok(d.out_bits), REPQ_INVALID_ARG, "qgemm: out_bits must be 4, 6 or 8");
    REPQ_REQUIRE(d.out_groups >= 1 && d.out_groups <= REPQ_MAX_OUT_GROUPS && d.N % d.out_groups == 0,
                 REPQ_INVALID_ARG, "qgemm: out_groups must be 1..4 and divide N");
    for (int g = 0; g < d.out_groups; ++g) {
      REPQ_REQUIRE(d.out_scale[g] > 0.f, REPQ_INVALID_ARG, "qgemm: out_scale[%d] must be positive", g);
      REPQ_REQUIRE(d.out_zero[g] > -(1 << 20) && d.out_zero[g] < (1 << 20), REPQ_INVALID_ARG, "qgemm: |out_zero| must be below 2^20");
    }
    REPQ_REQUIRE(d.ldo >= code_row_bytes(n_out, d.out_bits), REPQ_INVALID_ARG, "qgemm: ldo shorter than a row of codes");
    if (packed4(d.out_bits)) REPQ_REQUIRE((n_out / d.out_groups) % 2 == 0, REPQ_UNSUPPORTED, "qgemm: 4-bit output groups must have even width");
  } else {
    REPQ_REQUIRE(d.ldo >= n_out, REPQ_INVALID_ARG, "qgemm: ldo < output columns");
    const size_t esz = d.out_kind == REPQ_OUT_F32 ? 4 : 2;
    REPQ_REQUIRE(aligned(d.out, esz), REPQ_ALIGNMENT, "qgemm: out is not element-aligned");
  }
  if (d.residual) {
    REPQ_REQUIRE(d.residual_dtype == REPQ_F32 || d.residual_dtype == REPQ_BF16, REPQ_INVALID_ARG, "qgemm: residual_dtype");
    REPQ_REQUIRE(d.ld_residual >= d.N, REPQ_INVALID_ARG, "qgemm: ld_residual < N");
  }
  if (d.rope_cos_sin || d.glu) {
    REPQ_REQUIRE(!batched && !d.gelu && !d.residual, REPQ_UNSUPPORTED,
                 "qgemm: rope / glu are for plain products without gelu or residual");
    REPQ_REQUIRE(!(d.rope_cos_sin && d.glu), REPQ_UNSUPPORTED, "qgemm: rope and glu exclude each other");
    REPQ_REQUIRE(d.N % 2 == 0, REPQ_INVALID_ARG, "qgemm: rope / glu need an even N");
  }
  if (d.rope_cos_sin) {
    const int groups = d.out_groups >= 1 ? d.out_groups : 1;
    REPQ_REQUIRE(groups <= REPQ_MAX_OUT_GROUPS && d.N % groups == 0, REPQ_INVALID_ARG, "qgemm: out_groups must be 1..4 and divide N");
    REPQ_REQUIRE(d.rope_period > 0 && d.rope_dim > 0 && d.rope_dim % 16 == 0 && (d.N / groups) % d.rope_dim == 0,
                 REPQ_INVALID_ARG, "qgemm: rope_dim must be a multiple of 16 that divides N / out_groups, rope_period positive");
    REPQ_REQUIRE(d.rope_groups >= 1 && d.rope_groups <= groups, REPQ_INVALID_ARG, "qgemm: rope_groups must be 1..out_groups");
    REPQ_REQUIRE(aligned(d.rope_cos_sin, 16), REPQ_ALIGNMENT, "qgemm: rope_cos_sin must be 16-byte aligned");
  }
  return REPQ_OK;
}

EpilogueParams make_epilogue(const repq_gemm_desc& d) {
  EpilogueParams ep{};
  ep.s_w = d.s_w; ep.z_w = d.z_w; ep.s_w_scalar = d.s_w_scalar; ep.z_w_scalar = d.z_w_scalar;
  ep.bias = d.bias;
  ep.scale_a = d.alpha * d.s_a;
  ep.z_a = d.z_a; ep.K = d.K; ep.N = d.N;
  ep.gelu = d.gelu;
  ep.residual = d.residual; ep.residual_bf16 = d.residual_dtype == REPQ_BF16; ep.ld_residual = d.ld_residual;
  ep.out_kind = d.out_kind;
  const bool codes = d.out_kind == REPQ_OUT_CODES;
  ep.qmax = codes ? code_max(d.out_bits) : 0;
  ep.pack4 = codes && packed4(d.out_bits);
  ep.group_width = codes ? d.N / d.out_groups : d.N;
  for (int g = 0; g < REPQ_MAX_OUT_GROUPS; ++g) {
    const bool on = codes && g < d.out_groups;
    ep.inv_out_scale[g] = on ? 1.f / d.out_scale[g] : 1.f;
    ep.out_zero[g] = on ? d.out_zero[g] : 0;
  }
  ep.out = d.out; ep.ldo = d.ldo;
  ep.out_row_sum = codes ? d.out_row_sum : nullptr;
  ep.acc_debug = d.acc_debug;
  ep.rope = reinterpret_cast<const float2*>(d.rope_cos_sin);
  ep.rope_period = d.rope_period;
  ep.rope_dim = d.rope_dim;
  ep.rope_cols = d.rope_cos_sin ? d.rope_groups * (d.N / (d.out_groups >= 1 ? d.out_groups : 1)) : 0;
  ep.glu = d.glu;
  return ep;
}

}  // namespace

repq_status launch_row_sum(const uint8_t* codes, int bits, int64_t rows, int64_t n, int64_t ld_bytes,
                           int32_t* out, cudaStream_t st) {
  if (rows == 0) return REPQ_OK;
  const int64_t blocks = (rows + 7) / 8;
  const int grid = int(blocks < 4096 ? blocks : 4096);
  row_sum_kernel<<<grid, 256, 0, st>>>(codes, packed4(bits) ? 4 : packed6(bits) ? 6 : 8, rows, n, ld_bytes, out);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

repq_status launch_expand4(const uint8_t* src, int64_t rows, int64_t n, int64_t ld_src, uint8_t* dst,
                           int64_t ld_dst, int64_t n_pad, cudaStream_t st) {
  if (rows == 0) return REPQ_OK;
  const int64_t total = rows * (n_pad / 16);
  const int64_t blocks = (total + 255) / 256;
  const int grid = int(blocks < 8192 ? blocks : 8192);
  expand4_kernel<<<grid, 256, 0, st>>>(src, rows, n, ld_src, dst, ld_dst, n_pad);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace repq

using namespace repq;

extern "C" repq_status repq_qgemm_workspace_bytes(const repq_gemm_desc* d, size_t* bytes) {
  REPQ_REQUIRE(d && bytes, REPQ_INVALID_ARG, "qgemm_workspace_bytes: NULL argument");
  REPQ_TRY(validate(*d));
  *bytes = (d->M > 0 && !scores_supported(*d) && qgemm_tc_supported(*d)) ? qgemm_tc_workspace(*d) : 0;
  return REPQ_OK;
}

extern "C" repq_status repq_qgemm(const repq_gemm_desc* d, void* workspace, size_t workspace_bytes, void* stream) {
  REPQ_REQUIRE(d, REPQ_INVALID_ARG, "qgemm: NULL descriptor");
  REPQ_TRY(validate(*d));
  if (d->M == 0) return REPQ_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (scores_supported(*d)) return scores_tc_supported(*d) ? launch_scores_tc(*d, st) : launch_scores(*d, st);
  const EpilogueParams ep = make_epilogue(*d);
  if (qgemm_tc_supported(*d)) {
    const size_t need = qgemm_tc_workspace(*d);
    REPQ_REQUIRE(workspace_bytes >= need && (need == 0 || workspace), REPQ_WORKSPACE_TOO_SMALL,
                 "qgemm: workspace of %zu bytes given, %zu needed", workspace_bytes, need);
    return qgemm_tc(*d, ep, workspace, workspace_bytes, st);
  }
  return qgemm_mma(*d, ep, st);
}
