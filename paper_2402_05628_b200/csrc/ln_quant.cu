// Fused LayerNorm + layer-wise uniform quantization (Eq. 9 with the reparameterized affine factors of
// Eq. 12, then Eq. 4 with the scalar (s~, z~)).
//
// HBM-bound: every input element is read once with 128-bit loads and leaves as a 4-bit (or 8-bit)
// code.  A row is owned by a group of TPR threads; each thread keeps its slice of the row in
// registers, so mean and centred variance are two register passes with shuffle reductions.  The
// per-channel factors gamma~/s~ and beta~/s~ are loaded once per thread and reused for every row the
// thread processes (persistent grid-stride loop over rows).
#include <cuda_bf16.h>

#include "common.h"

namespace repq {
namespace {

constexpr int kChunk = 8;   // elements per 128-bit bf16 load
constexpr int kVPT = 4;     // chunks per thread (upper bound)

__device__ __forceinline__ void load_chunk(const float* p, float (&v)[kChunk]) {
  const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ void load_chunk(const __nv_bfloat16* p, float (&v)[kChunk]) {
  const uint4 a = __ldcs(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

template <int TPR, typename V>
__device__ __forceinline__ V group_reduce(V v, V* red, int group_first_warp) {
  constexpr int kShfl = TPR < 32 ? TPR : 32;
#pragma unroll
  for (int o = kShfl / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if constexpr (TPR > 32) {
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    v = V(0);
#pragma unroll
    for (int w = 0; w < TPR / 32; ++w) v += red[group_first_warp + w];
  }
  return v;
}

template <typename T, int TPR, bool kPack4>
__global__ void __launch_bounds__((TPR > 256 ? TPR : 256))
ln_quant_kernel(const T* __restrict__ x, int64_t rows, int D, int64_t ldx,
                const float* __restrict__ gamma_t, const float* __restrict__ beta_t, float eps, int rms,
                float inv_s, int z, int qmax, uint8_t* __restrict__ codes, int64_t ldc,
                int32_t* __restrict__ row_sum) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR;
  // one array per reduction of a row: a thread can only overwrite an array after every thread of the
  // block has passed the barrier of a later reduction, hence has finished reading it
  __shared__ float red_a[kBlock / 32];
  __shared__ float red_b[kBlock / 32];
  __shared__ int red_c[kBlock / 32];

  const int tig = threadIdx.x % TPR;             // thread in group
  const int group = threadIdx.x / TPR;
  const int group_first_warp = (group * TPR) >> 5;
  const int nchunks = D / kChunk;

  // per-channel factors, pre-divided by the layer-wise scale: t = xhat * g + b = y / s~
  float g[kVPT][kChunk], b[kVPT][kChunk];
#pragma unroll
  for (int i = 0; i < kVPT; ++i) {
    const int c = tig + i * TPR;
    if (c < nchunks) {
#pragma unroll
      for (int e = 0; e < kChunk; ++e) {
        g[i][e] = __ldg(gamma_t + c * kChunk + e) * inv_s;
        b[i][e] = __ldg(beta_t + c * kChunk + e) * inv_s;
      }
    }
  }
  const float t_lo = float(-z), t_hi = float(qmax - z);
  const float inv_d = 1.f / float(D);

  for (int64_t base = int64_t(blockIdx.x) * kRowsPerBlock; base < rows;
       base += int64_t(gridDim.x) * kRowsPerBlock) {
    const int64_t row = base + group;
    const bool live = row < rows;
    const T* xr = x + (live ? row : 0) * ldx;

    float v[kVPT][kChunk];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int c = tig + i * TPR;
      if (c < nchunks && live) {
        load_chunk(xr + c * kChunk, v[i]);
#pragma unroll
        for (int e = 0; e < kChunk; ++e) sum += v[i][e];
      } else {
#pragma unroll
        for (int e = 0; e < kChunk; ++e) v[i][e] = 0.f;
      }
    }
    float mu = 0.f;
    if (!rms) mu = group_reduce<TPR, float>(sum, red_a, group_first_warp) * inv_d;

    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int c = tig + i * TPR;
      if (c < nchunks) {
#pragma unroll
        for (int e = 0; e < kChunk; ++e) {
          v[i][e] -= mu;
          ss = fmaf(v[i][e], v[i][e], ss);
        }
      }
    }
    const float var = group_reduce<TPR, float>(ss, red_b, group_first_warp) * inv_d;
    const float rstd = rsqrtf(var + eps);

    int csum = 0;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int c = tig + i * TPR;
      if (c < nchunks) {
        int q[kChunk];
#pragma unroll
        for (int e = 0; e < kChunk; ++e) {
          float t = fmaf(v[i][e] * rstd, g[i][e], b[i][e]);
          t = fminf(fmaxf(t, t_lo), t_hi);        // clip(round(t) + z, 0, qmax) == round(clamp(t)) + z
          q[e] = __float2int_rn(t) + z;
          csum += q[e];
        }
        if (live) {
          uint8_t* out = codes + row * ldc;
          if constexpr (kPack4) {
            uint32_t w = 0;
#pragma unroll
            for (int e = 0; e < kChunk; ++e) w |= uint32_t(q[e]) << (4 * e);
            reinterpret_cast<uint32_t*>(out)[c] = w;
          } else {
            uint2 w;
            w.x = uint32_t(q[0]) | uint32_t(q[1]) << 8 | uint32_t(q[2]) << 16 | uint32_t(q[3]) << 24;
            w.y = uint32_t(q[4]) | uint32_t(q[5]) << 8 | uint32_t(q[6]) << 16 | uint32_t(q[7]) << 24;
            reinterpret_cast<uint2*>(out)[c] = w;
          }
        }
      }
    }
    if (row_sum != nullptr) {
      csum = group_reduce<TPR, int>(csum, red_c, group_first_warp);
      if (live && tig == 0) row_sum[row] = csum;
    }
  }
}

template <typename T, int TPR>
repq_status launch(const T* x, int64_t rows, int D, int64_t ldx, const float* g, const float* b, float eps,
                   int rms, float s_t, int z, int bits, uint8_t* codes, int64_t ldc, int32_t* row_sum,
                   cudaStream_t st) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR;
  const int64_t need = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
  const int64_t cap = int64_t(sm_count()) * 8;
  const int grid = int(need < cap ? need : cap);
  const float inv_s = 1.f / s_t;
  const int qmax = (1 << bits) - 1;
  if (bits == 4)
    ln_quant_kernel<T, TPR, true><<<grid, kBlock, 0, st>>>(x, rows, D, ldx, g, b, eps, rms, inv_s, z, qmax, codes, ldc, row_sum);
  else
    ln_quant_kernel<T, TPR, false><<<grid, kBlock, 0, st>>>(x, rows, D, ldx, g, b, eps, rms, inv_s, z, qmax, codes, ldc, row_sum);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

template <typename T>
repq_status dispatch(const T* x, int64_t rows, int D, int64_t ldx, const float* g, const float* b, float eps,
                     int rms, float s_t, int z, int bits, uint8_t* codes, int64_t ldc, int32_t* row_sum,
                     cudaStream_t st) {
  const int nchunks = D / kChunk;
#define REPQ_LN_CASE(TPR) \
  if (nchunks <= TPR * kVPT) return launch<T, TPR>(x, rows, D, ldx, g, b, eps, rms, s_t, z, bits, codes, ldc, row_sum, st);
  REPQ_LN_CASE(8)
  REPQ_LN_CASE(16)
  REPQ_LN_CASE(32)
  REPQ_LN_CASE(64)
  REPQ_LN_CASE(128)
  REPQ_LN_CASE(256)
  REPQ_LN_CASE(512)
#undef REPQ_LN_CASE
  return fail(REPQ_UNSUPPORTED, "ln_quant: D = %d exceeds 16384", D);
}

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_ln_quant(const void* x, int x_dtype, int64_t rows, int D, int64_t ldx,
                                     const float* gamma_t, const float* beta_t, float eps, int norm_kind,
                                     float s_t, int z_t, int bits, uint8_t* codes, int64_t ld_codes_bytes,
                                     int32_t* row_sum, void* stream) {
  REPQ_REQUIRE(rows >= 0 && D > 0, REPQ_INVALID_ARG, "ln_quant: rows must be >= 0 and D > 0");
  if (rows == 0) return REPQ_OK;
  REPQ_REQUIRE(x && gamma_t && beta_t && codes, REPQ_INVALID_ARG, "ln_quant: NULL pointer");
  REPQ_REQUIRE(x_dtype == REPQ_F32 || x_dtype == REPQ_BF16, REPQ_INVALID_ARG, "ln_quant: x_dtype must be REPQ_F32 or REPQ_BF16");
  REPQ_REQUIRE(norm_kind == REPQ_NORM_LAYERNORM || norm_kind == REPQ_NORM_RMS, REPQ_INVALID_ARG, "ln_quant: unknown norm_kind");
  REPQ_REQUIRE(bits_ok(bits), REPQ_INVALID_ARG, "ln_quant: bits must be 4, 6 or 8");
  REPQ_REQUIRE(s_t > 0.f && eps >= 0.f, REPQ_INVALID_ARG, "ln_quant: s_t must be positive and eps non-negative");
  REPQ_REQUIRE(z_t > -(1 << 20) && z_t < (1 << 20), REPQ_INVALID_ARG, "ln_quant: |z_t| must be below 2^20");
  REPQ_REQUIRE(D % 8 == 0, REPQ_UNSUPPORTED, "ln_quant: D = %d must be a multiple of 8", D);
  REPQ_REQUIRE(D <= 16384, REPQ_UNSUPPORTED, "ln_quant: D = %d exceeds 16384", D);
  REPQ_REQUIRE(ldx >= D, REPQ_INVALID_ARG, "ln_quant: ldx < D");
  const size_t esz = x_dtype == REPQ_F32 ? 4 : 2;
  REPQ_REQUIRE(aligned(x, 16) && (size_t(ldx) * esz) % 16 == 0, REPQ_ALIGNMENT, "ln_quant: x rows must be 16-byte aligned");
  const int64_t unit = bits == 4 ? 4 : 8;
  REPQ_REQUIRE(ld_codes_bytes >= code_row_bytes(D, bits), REPQ_INVALID_ARG, "ln_quant: ld_codes_bytes shorter than a row");
  REPQ_REQUIRE(aligned(codes, unit) && ld_codes_bytes % unit == 0, REPQ_ALIGNMENT,
               "ln_quant: codes rows must be %d-byte aligned", int(unit));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rms = norm_kind == REPQ_NORM_RMS;
  if (x_dtype == REPQ_F32)
    return dispatch(static_cast<const float*>(x), rows, D, ldx, gamma_t, beta_t, eps, rms, s_t, z_t, bits, codes, ld_codes_bytes, row_sum, st);
  return dispatch(static_cast<const __nv_bfloat16*>(x), rows, D, ldx, gamma_t, beta_t, eps, rms, s_t, z_t, bits, codes, ld_codes_bytes, row_sum, st);
}
