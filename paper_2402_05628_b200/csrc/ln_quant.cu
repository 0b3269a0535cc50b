// Fused LayerNorm + layer-wise uniform quantization (Eq. 9 with the reparameterized affine factors of
// Eq. 12, then Eq. 4 with the scalar (s~, z~)).
//
// HBM-bound: every input element is read once with 128-bit loads and leaves as a 4-bit (or 8-bit)
// code.  A row is owned by a group of TPR threads which keeps its slice of the row in registers, so mean
// and centred variance are two register passes with shuffle reductions.  Each group works on kRows rows
// at a time (all their loads are issued before the first reduction) to keep enough bytes in flight.
// The per-channel factors gamma~/s~ and beta~/s~ are staged once per CTA in shared memory.
//
// Rounding: round_half_even(clamp(t, -z, qmax - z)) is taken with one float add of 1.5 * 2^23 (the float
// adder rounds to nearest-even at integer granularity there, with the tie decided by the parity of the
// rounded t itself, as Eq. 4 has it); the integer then sits in the low mantissa bits and z is added while
// the codes are packed.
#include <cuda_bf16.h>

#include "common.h"

namespace repq {
namespace {

constexpr int kChunk = 8;   // elements per 128-bit bf16 load
constexpr int kVPT = 4;     // chunks per thread (upper bound)
constexpr int kRows = 2;    // rows in flight per thread group
constexpr uint32_t kMagicBits = 0x4B400000u;   // 1.5 * 2^23

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

// Sum over the TPR threads of a group, for kRows values at once.
template <int TPR, typename V>
__device__ __forceinline__ void group_reduce(V (&v)[kRows], V* red, int group_first_warp) {
  constexpr int kShfl = TPR < 32 ? TPR : 32;
#pragma unroll
  for (int o = kShfl / 2; o > 0; o >>= 1)
#pragma unroll
    for (int r = 0; r < kRows; ++r) v[r] += __shfl_xor_sync(0xffffffffu, v[r], o);
  if constexpr (TPR > 32) {
    if ((threadIdx.x & 31) == 0)
#pragma unroll
      for (int r = 0; r < kRows; ++r) red[(threadIdx.x >> 5) * kRows + r] = v[r];
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      V acc = V(0);
#pragma unroll
      for (int w = 0; w < TPR / 32; ++w) acc += red[(group_first_warp + w) * kRows + r];
      v[r] = acc;
    }
  }
}

template <typename T, int TPR, bool kPack4>
__global__ void __launch_bounds__((TPR > 256 ? TPR : 256))
ln_quant_kernel(const T* __restrict__ x, int64_t rows, int D, int64_t ldx,
                const float* __restrict__ gamma_t, const float* __restrict__ beta_t, float eps, int rms,
                float inv_s, int z, int qmax, uint8_t* __restrict__ codes, int64_t ldc,
                int32_t* __restrict__ row_sum) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kGroups = kBlock / TPR;
  constexpr int kRowsPerBlock = kGroups * kRows;
  extern __shared__ __align__(16) float s_gb[];          // g[D] then b[D]: gamma~/s~ and beta~/s~
  // one array per reduction of a row: it can only be overwritten after every thread of the block has
  // passed the barrier of a later reduction, hence has finished reading it
  __shared__ float red_a[kBlock / 32 * kRows];
  __shared__ float red_b[kBlock / 32 * kRows];
  __shared__ int red_c[kBlock / 32 * kRows];

  float* s_g = s_gb;
  float* s_b = s_gb + D;
  for (int i = threadIdx.x; i < D; i += kBlock) {
    s_g[i] = __ldg(gamma_t + i) * inv_s;
    s_b[i] = __ldg(beta_t + i) * inv_s;
  }
  __syncthreads();

  const int tig = threadIdx.x % TPR;             // thread in group
  const int group = threadIdx.x / TPR;
  const int group_first_warp = (group * TPR) >> 5;
  const int nchunks = D / kChunk;
  const float t_lo = float(-z), t_hi = float(qmax - z);
  const float magic = __uint_as_float(kMagicBits);
  const float inv_d = 1.f / float(D);

  for (int64_t base = int64_t(blockIdx.x) * kRowsPerBlock; base < rows;
       base += int64_t(gridDim.x) * kRowsPerBlock) {
    const int64_t row0 = base + group * kRows;

    float v[kRows][kVPT][kChunk];
    float sum[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const bool live = row0 + r < rows;
      const T* xr = x + (live ? row0 + r : 0) * ldx;
      sum[r] = 0.f;
#pragma unroll
      for (int i = 0; i < kVPT; ++i) {
        const int c = tig + i * TPR;
        if (c < nchunks && live) {
          load_chunk(xr + c * kChunk, v[r][i]);
        } else {
#pragma unroll
          for (int e = 0; e < kChunk; ++e) v[r][i][e] = 0.f;
        }
      }
    }
#pragma unroll
    for (int r = 0; r < kRows; ++r)
#pragma unroll
      for (int i = 0; i < kVPT; ++i)
#pragma unroll
        for (int e = 0; e < kChunk; ++e) sum[r] += v[r][i][e];

    float mu[kRows];
    if (!rms) {
      group_reduce<TPR, float>(sum, red_a, group_first_warp);
#pragma unroll
      for (int r = 0; r < kRows; ++r) mu[r] = sum[r] * inv_d;
    } else {
#pragma unroll
      for (int r = 0; r < kRows; ++r) mu[r] = 0.f;
    }

    float ss[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      ss[r] = 0.f;
#pragma unroll
      for (int i = 0; i < kVPT; ++i) {
        if (tig + i * TPR < nchunks) {
#pragma unroll
          for (int e = 0; e < kChunk; ++e) {
            v[r][i][e] -= mu[r];
            ss[r] = fmaf(v[r][i][e], v[r][i][e], ss[r]);
          }
        }
      }
    }
    group_reduce<TPR, float>(ss, red_b, group_first_warp);
    float rstd[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) rstd[r] = rsqrtf(ss[r] * inv_d + eps);

    int csum[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) csum[r] = 0;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int c = tig + i * TPR;
      if (c < nchunks) {
        float g[kChunk], b[kChunk];
        {
          const float4 g0 = *reinterpret_cast<const float4*>(s_g + c * kChunk);
          const float4 g1 = *reinterpret_cast<const float4*>(s_g + c * kChunk + 4);
          const float4 b0 = *reinterpret_cast<const float4*>(s_b + c * kChunk);
          const float4 b1 = *reinterpret_cast<const float4*>(s_b + c * kChunk + 4);
          g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w; g[4] = g1.x; g[5] = g1.y; g[6] = g1.z; g[7] = g1.w;
          b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w; b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
          uint32_t u[kChunk];
#pragma unroll
          for (int e = 0; e < kChunk; ++e) {
            float t = fmaf(v[r][i][e] * rstd[r], g[e], b[e]);
            t = fminf(fmaxf(t, t_lo), t_hi);       // clip(round(t) + z, 0, qmax) == round(clamp(t)) + z
            u[e] = __float_as_uint(t + magic);     // = magic_bits + round_half_even(t), as integers
          }
          if (row0 + r < rows) {
            uint8_t* out = codes + (row0 + r) * ldc;
            if constexpr (kPack4) {
              // sum_e (magic_bits + round(t_e)) << 4e  -  sum_e (magic_bits - z) << 4e  =  sum_e code_e << 4e
              uint32_t w = 0;
#pragma unroll
              for (int e = 0; e < kChunk; ++e) w += u[e] << (4 * e);
              uint32_t k = 0;
#pragma unroll
              for (int e = 0; e < kChunk; ++e) k += (kMagicBits - uint32_t(z)) << (4 * e);
              w -= k;
              reinterpret_cast<uint32_t*>(out)[c] = w;
              csum[r] += __dp4a(w & 0x0F0F0F0Fu, 0x01010101u, 0u) + __dp4a((w >> 4) & 0x0F0F0F0Fu, 0x01010101u, 0u);
            } else {
              uint2 w;
              // low bytes hold round(t_e) mod 256; a per-byte add of z gives the codes (all in [0, 255])
              const uint32_t z4 = (uint32_t(z) & 0xFFu) * 0x01010101u;
              w.x = __vadd4(__byte_perm(__byte_perm(u[0], u[1], 0x0040), __byte_perm(u[2], u[3], 0x0040), 0x5410), z4);
              w.y = __vadd4(__byte_perm(__byte_perm(u[4], u[5], 0x0040), __byte_perm(u[6], u[7], 0x0040), 0x5410), z4);
              reinterpret_cast<uint2*>(out)[c] = w;
              csum[r] += __dp4a(w.x, 0x01010101u, 0u) + __dp4a(w.y, 0x01010101u, 0u);
            }
          }
        }
      }
    }
    if (row_sum != nullptr) {
      group_reduce<TPR, int>(csum, red_c, group_first_warp);
      if (tig == 0) {
#pragma unroll
        for (int r = 0; r < kRows; ++r)
          if (row0 + r < rows) row_sum[row0 + r] = csum[r];
      }
    }
  }
}

template <typename T, int TPR>
repq_status launch(const T* x, int64_t rows, int D, int64_t ldx, const float* g, const float* b, float eps,
                   int rms, float s_t, int z, int bits, uint8_t* codes, int64_t ldc, int32_t* row_sum,
                   cudaStream_t st) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR * kRows;
  const int64_t need = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
  const int64_t cap = int64_t(sm_count()) * 8;
  const int grid = int(need < cap ? need : cap);
  const float inv_s = 1.f / s_t;
  const int qmax = code_max(bits);
  const size_t smem = size_t(D) * 2 * sizeof(float);
  auto kern = packed4(bits) ? ln_quant_kernel<T, TPR, true> : ln_quant_kernel<T, TPR, false>;
  if (smem > 48 * 1024) REPQ_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  kern<<<grid, kBlock, smem, st>>>(x, rows, D, ldx, g, b, eps, rms, inv_s, z, qmax, codes, ldc, row_sum);
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
  const int64_t unit = packed4(bits) ? 4 : 8;
  REPQ_REQUIRE(ld_codes_bytes >= code_row_bytes(D, bits), REPQ_INVALID_ARG, "ln_quant: ld_codes_bytes shorter than a row");
  REPQ_REQUIRE(aligned(codes, unit) && ld_codes_bytes % unit == 0, REPQ_ALIGNMENT,
               "ln_quant: codes rows must be %d-byte aligned", int(unit));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rms = norm_kind == REPQ_NORM_RMS;
  if (x_dtype == REPQ_F32)
    return dispatch(static_cast<const float*>(x), rows, D, ldx, gamma_t, beta_t, eps, rms, s_t, z_t, bits, codes, ld_codes_bytes, row_sum, st);
  return dispatch(static_cast<const __nv_bfloat16*>(x), rows, D, ldx, gamma_t, beta_t, eps, rms, s_t, z_t, bits, codes, ld_codes_bytes, row_sum, st);
}
