// Shared GEMM epilogue: zero-point correction, de-quantization, bias, GELU, residual, and the optional
// re-quantization of Eq. 4.  Used by both the tensor-memory GEMM and the warp-MMA GEMM so that the two
// produce identical results.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

#include "../../include/repq.h"
#include "f32x2.cuh"

namespace repq {

struct EpilogueParams {
  const float* s_w;        // per output channel or nullptr
  const int32_t* z_w;      // per output channel or nullptr
  float s_w_scalar;
  int32_t z_w_scalar;
  const float* bias;       // or nullptr
  float scale_a;           // alpha * s_a
  int32_t z_a;
  int32_t K;
  int32_t N;
  int32_t gelu;
  const void* residual;    // or nullptr
  int32_t residual_bf16;
  int64_t ld_residual;
  int32_t out_kind;
  int32_t qmax;            // 2^out_bits - 1
  int32_t pack4;           // out_bits == 4
  int32_t group_width;     // N / out_groups
  float inv_out_scale[REPQ_MAX_OUT_GROUPS];
  int32_t out_zero[REPQ_MAX_OUT_GROUPS];
  void* out;
  int64_t ldo;
  int32_t* out_row_sum;    // or nullptr
  int32_t* acc_debug;      // or nullptr, dense M x N
  // steps on pairs of neighbouring columns (LLaMA block form), applied to v before the output conversion
  const float2* rope;      // (cos, sin) table [rope_period][rope_dim / 2], or nullptr
  int32_t rope_period;
  int32_t rope_dim;
  int32_t rope_cols;       // columns below this bound are rotated
  int32_t glu;             // columns (2i, 2i+1) = (gate, up): output column i = silu(gate) * up
};

// Per-column constants of the epilogue, gathered once per output column.
struct ColumnTerms {
  float scale;    // alpha * s_a * s_w[j]
  float bias;
  int32_t z_w;
  int32_t kzz;    // K * z_a * z_w[j] - z_a * wsum[j]
  float inv_so;
  float zo_lo, zo_hi;
  int32_t zo;
};

__device__ __forceinline__ ColumnTerms column_terms(const EpilogueParams& p, int j, int32_t wsum_j) {
  ColumnTerms c;
  const float sw = p.s_w ? __ldg(p.s_w + j) : p.s_w_scalar;
  c.z_w = p.z_w ? __ldg(p.z_w + j) : p.z_w_scalar;
  c.scale = p.scale_a * sw;
  c.bias = p.bias ? __ldg(p.bias + j) : 0.f;
  // wrap-around integer arithmetic: only the final correction has to fit 32 bits
  c.kzz = int32_t(uint32_t(p.K) * uint32_t(p.z_a) * uint32_t(c.z_w) - uint32_t(p.z_a) * uint32_t(wsum_j));
  const int g = p.out_kind == REPQ_OUT_CODES ? j / p.group_width : 0;
  c.inv_so = p.inv_out_scale[g];
  c.zo = p.out_zero[g];
  c.zo_lo = float(-c.zo);
  c.zo_hi = float(p.qmax - c.zo);
  return c;
}

// erf-form GELU, v * Phi(v), without branches.  With t = |v| / sqrt2 clamped to 4 (erfc(4) < 2e-8),
//     erfc(t) = 2^(-t q(t)),   Phi(v) = h for v < 0,   1 - h otherwise,   h = erfc(t) / 2 = 2^(-t q(t) - 1),
// and q, which is smooth (q(0) = 2 / (sqrt(pi) ln 2), q(t) ~ t / ln 2), is a degree-6 polynomial fitted so that
// the error of erf stays below 1e-7.  The negative tail keeps its relative accuracy (no 1 + erf cancellation).
// Against the float64 erf form the float32 result is within 1.4e-7 |v| (about one ulp).
__device__ __forceinline__ float gelu_erf(float v) {
  const float t = fminf(fabsf(v) * 0.70710678118654752f, 4.f);
  float q = -1.002269491e-04f;
  q = fmaf(q, t, 4.616116930e-04f);
  q = fmaf(q, t, 2.302142326e-03f);
  q = fmaf(q, t, -2.945240214e-02f);
  q = fmaf(q, t, 1.489636004e-01f);
  q = fmaf(q, t, 9.183286428e-01f);
  q = fmaf(q, t, 1.627913713e+00f);
  float h;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(h) : "f"(fmaf(-t, q, -1.f)));
  return v * (v < 0.f ? h : 1.f - h);
}

// The same on two values at once (packed float pairs where the operation exists in that form): every lane goes through
// the operations of gelu_erf in the same order, so the results are the same bits.
__device__ __forceinline__ void gelu_erf_pair(float& v0, float& v1) {
  float a0, a1;
  unpack2(mul2(pack2(v0, v1), splat2(0.70710678118654752f)), a0, a1);       // |v| c = |v c|
  const f32x2 t = pack2(fminf(fabsf(a0), 4.f), fminf(fabsf(a1), 4.f));
  f32x2 q = splat2(-1.002269491e-04f);
  q = fma2(q, t, splat2(4.616116930e-04f));
  q = fma2(q, t, splat2(2.302142326e-03f));
  q = fma2(q, t, splat2(-2.945240214e-02f));
  q = fma2(q, t, splat2(1.489636004e-01f));
  q = fma2(q, t, splat2(9.183286428e-01f));
  q = fma2(q, t, splat2(1.627913713e+00f));
  float e0, e1, h0, h1;
  unpack2(fma2(t, q, splat2(1.f)), e0, e1);                                  // fma(-t, q, -1) = -fma(t, q, 1)
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(h0) : "f"(-e0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(h1) : "f"(-e1));
  unpack2(mul2(pack2(v0, v1), pack2(v0 < 0.f ? h0 : 1.f - h0, v1 < 0.f ? h1 : 1.f - h1)), v0, v1);
}

// acc -> corrected integer -> float value before the output conversion.
__device__ __forceinline__ float epilogue_value(const EpilogueParams& p, const ColumnTerms& c, int32_t acc,
                                                int32_t asum_m, int64_t m, int j) {
  const int32_t corr = int32_t(uint32_t(acc) - uint32_t(c.z_w) * uint32_t(asum_m) + uint32_t(c.kzz));
  float v = fmaf(c.scale, float(corr), c.bias);
  if (p.gelu) v = gelu_erf(v);
  if (p.residual) {
    const int64_t off = m * p.ld_residual + j;
    v += p.residual_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(p.residual)[off])
                         : static_cast<const float*>(p.residual)[off];
  }
  return v;
}

// Rotary position embedding of one pair: (a, b) at column pair index `pair` of its head, row position `pos`.
__device__ __forceinline__ void rope_rotate(const float2 cs, float& a, float& b) {
  const float ra = fmaf(a, cs.x, -(b * cs.y));
  const float rb = fmaf(a, cs.y, b * cs.x);
  a = ra;
  b = rb;
}

// silu(g) * u, silu(x) = x / (1 + exp(-x)); exp(-x) = +inf for very negative x gives -0 * u.
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

// Eq. 4 with the output quantizer: clip(round(v / s_o) + z_o, 0, qmax).
__device__ __forceinline__ int32_t requantize(const ColumnTerms& c, float v) {
  float t = v * c.inv_so;
  t = fminf(fmaxf(t, c.zo_lo), c.zo_hi);
  return __float2int_rn(t) + c.zo;
}

}  // namespace repq
