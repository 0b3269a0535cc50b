// Integer GEMM on warp-level MMA (m16n8k32, u8 x u8 -> s32) for shapes the tensor-memory kernel does
// not take: batched code-by-code products (attention scores per (batch, head)), small or ragged
// problems, unaligned strides.  4-bit operands are expanded to bytes while they are copied to shared
// memory; operand row sums for the zero-point correction are accumulated by the same copy.
#include "common.h"
#include "epilogue.cuh"
#include "kernels.h"

namespace repq {
namespace {

constexpr int BM = 64, BN = 64, BK = 64;     // CTA tile (BK in codes = bytes after expansion)
constexpr int kThreads = 128;                // 4 warps, each 32 x 32 of the tile
constexpr int kRowBytes = BK + 16;           // padded shared-memory row: conflict-free fragment loads
constexpr int kWordsPerRow = BK / 4;

struct MmaOperand {
  const uint8_t* base;
  int64_t ld;
  int rows;        // valid rows of this operand (M or N)
  int bits;
};

// Returns 4 consecutive codes (one per byte) starting at code index k0 (multiple of 4) of a row, zero
// beyond K.  `aligned4` says base and ld allow 32-bit / 16-bit loads at these offsets.
__device__ __forceinline__ uint32_t load_codes4(const uint8_t* row, int k0, int K, int bits, bool aligned4) {
  if (k0 >= K) return 0u;
  if (bits == 6) {
    // four codes in three bytes: the 24 bits at byte 3 k0 / 4 of the row
    const uint8_t* p = row + (k0 >> 2) * 3;
    const int left = K - k0;
    uint32_t f = p[0];
    if (left > 1) f |= uint32_t(p[1]) << 8;
    if (left > 2) f |= uint32_t(p[2]) << 16;
    uint32_t r = (f & 0x3Fu) | ((f & 0xFC0u) << 2) | ((f & 0x3F000u) << 4) | ((f & 0xFC0000u) << 6);
    if (left < 4) r &= (1u << (8 * left)) - 1u;
    return r;
  }
  if (bits == 4) {
    const uint8_t* p = row + (k0 >> 1);
    uint32_t w;
    if (aligned4 && k0 + 4 <= K) {
      w = *reinterpret_cast<const uint16_t*>(p);
    } else {
      w = p[0];
      if (k0 + 2 < K) w |= uint32_t(p[1]) << 8;
    }
    // bytes b0 b1 -> codes (b0 & 15, b0 >> 4, b1 & 15, b1 >> 4)
    uint32_t r = (w & 0xF) | ((w & 0xF0) << 4) | ((w & 0xF00) << 8) | ((w & 0xF000) << 12);
    const int left = K - k0;
    if (left < 4) r &= (1u << (8 * left)) - 1u;
    return r;
  }
  if (aligned4 && k0 + 4 <= K) return *reinterpret_cast<const uint32_t*>(row + k0);
  uint32_t r = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (k0 + e < K) r |= uint32_t(row[k0 + e]) << (8 * e);
  return r;
}

__device__ __forceinline__ void mma_u8(int (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__global__ void __launch_bounds__(kThreads)
qgemm_mma_kernel(MmaOperand A, MmaOperand W, int K, int batch_inner, int64_t a_so, int64_t a_si, int64_t w_so,
                 int64_t w_si, int64_t o_so, int64_t o_si, bool a_al, bool w_al, EpilogueParams ep) {
  __shared__ __align__(16) uint8_t sA[BM * kRowBytes];
  __shared__ __align__(16) uint8_t sW[BN * kRowBytes];
  __shared__ int s_asum[BM];
  __shared__ int s_wsum[BN];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bo = blockIdx.z / batch_inner, bi = blockIdx.z % batch_inner;
  const uint8_t* a_base = A.base + bo * a_so + bi * a_si;
  const uint8_t* w_base = W.base + bo * w_so + bi * w_si;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;

  if (tid < BM) s_asum[tid] = 0;
  if (tid < BN) s_wsum[tid] = 0;

  // loader mapping: word w of the tile -> row w / 16, word-in-row w % 16; a thread keeps its rows
  constexpr int kLoads = BM * kWordsPerRow / kThreads;   // 8
  int a_part[kLoads], w_part[kLoads];
#pragma unroll
  for (int i = 0; i < kLoads; ++i) a_part[i] = w_part[i] = 0;

  const int wm = (warp >> 1) * 32, wn = (warp & 1) * 32;
  const int g = lane >> 2, t = lane & 3;
  int acc[2][4][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0;

  for (int k0 = 0; k0 < K; k0 += BK) {
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kLoads; ++i) {
      const int w = tid + i * kThreads;
      const int r = w / kWordsPerRow, c = w % kWordsPerRow;
      uint32_t va = 0, vw = 0;
      if (m0 + r < A.rows) va = load_codes4(a_base + int64_t(m0 + r) * A.ld, k0 + 4 * c, K, A.bits, a_al);
      if (n0 + r < W.rows) vw = load_codes4(w_base + int64_t(n0 + r) * W.ld, k0 + 4 * c, K, W.bits, w_al);
      *reinterpret_cast<uint32_t*>(sA + r * kRowBytes + 4 * c) = va;
      *reinterpret_cast<uint32_t*>(sW + r * kRowBytes + 4 * c) = vw;
      a_part[i] = __dp4a(va, 0x01010101u, uint32_t(a_part[i]));
      w_part[i] = __dp4a(vw, 0x01010101u, uint32_t(w_part[i]));
    }
    __syncthreads();
#pragma unroll
    for (int ks = 0; ks < BK; ks += 32) {
      uint32_t af[2][4], bf[4][2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint8_t* p = sA + (wm + i * 16 + g) * kRowBytes + ks + 4 * t;
        af[i][0] = *reinterpret_cast<const uint32_t*>(p);
        af[i][1] = *reinterpret_cast<const uint32_t*>(p + 8 * kRowBytes);
        af[i][2] = *reinterpret_cast<const uint32_t*>(p + 16);
        af[i][3] = *reinterpret_cast<const uint32_t*>(p + 8 * kRowBytes + 16);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint8_t* p = sW + (wn + j * 8 + g) * kRowBytes + ks + 4 * t;
        bf[j][0] = *reinterpret_cast<const uint32_t*>(p);
        bf[j][1] = *reinterpret_cast<const uint32_t*>(p + 16);
      }
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_u8(acc[i][j], af[i], bf[j]);
    }
  }

  // operand row sums
#pragma unroll
  for (int i = 0; i < kLoads; ++i) {
    const int r = (tid + i * kThreads) / kWordsPerRow;
    atomicAdd(&s_asum[r], a_part[i]);
    atomicAdd(&s_wsum[r], w_part[i]);
  }
  __syncthreads();

  // epilogue: thread holds rows (g, g + 8) and columns (2t, 2t + 1) of every 16 x 8 fragment
  if (ep.out_kind == REPQ_OUT_CODES) {
    ep.out = static_cast<uint8_t*>(ep.out) + bo * o_so + bi * o_si;
  } else if (ep.out_kind == REPQ_OUT_F32) {
    ep.out = static_cast<float*>(ep.out) + bo * o_so + bi * o_si;
  } else {
    ep.out = static_cast<__nv_bfloat16*>(ep.out) + bo * o_so + bi * o_si;
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int rl = wm + i * 16 + g + 8 * h;
      const int64_t m = m0 + rl;
      const bool row_ok = m < A.rows;
      const int asum_m = s_asum[rl];
      int code_sum = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int cl = wn + j * 8 + 2 * t;
        const int col = n0 + cl;
        int q[2] = {0, 0};
        float v[2] = {0.f, 0.f};
        ColumnTerms ct[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int jcol = col + e;
          if (row_ok && jcol < ep.N) {
            ct[e] = column_terms(ep, jcol, s_wsum[cl + e]);
            const int a = acc[i][j][2 * h + e];
            if (ep.acc_debug) ep.acc_debug[m * ep.N + jcol] = a;
            v[e] = epilogue_value(ep, ct[e], a, asum_m, m, jcol);
          }
        }
        // steps on the column pair (col is even, N is even when they are on)
        if (ep.rope != nullptr && row_ok && col < ep.rope_cols)
          rope_rotate(ep.rope[int64_t(m % ep.rope_period) * (ep.rope_dim >> 1) + ((col % ep.rope_dim) >> 1)], v[0], v[1]);
        if (ep.glu) {
          if (row_ok && col < ep.N) {
            const float hv = silu_mul(v[0], v[1]);
            const int oc = col >> 1;
            if (ep.out_kind == REPQ_OUT_F32) {
              static_cast<float*>(ep.out)[m * ep.ldo + oc] = hv;
            } else if (ep.out_kind == REPQ_OUT_BF16) {
              static_cast<__nv_bfloat16*>(ep.out)[m * ep.ldo + oc] = __float2bfloat16_rn(hv);
            } else {
              const int code = requantize(column_terms(ep, 0, 0), hv);     // one output group: its quantizer
              code_sum += code;
              static_cast<uint8_t*>(ep.out)[m * ep.ldo + oc] = uint8_t(code);
            }
          }
          continue;
        }
        if (ep.out_kind == REPQ_OUT_CODES) {
#pragma unroll
          for (int e = 0; e < 2; ++e)
            if (row_ok && col + e < ep.N) {
              q[e] = requantize(ct[e], v[e]);
              code_sum += q[e];
            }
        }
        if (row_ok && col < ep.N) {
          const bool two = col + 1 < ep.N;
          if (ep.out_kind == REPQ_OUT_F32) {
            float* o = static_cast<float*>(ep.out) + m * ep.ldo + col;
            o[0] = v[0];
            if (two) o[1] = v[1];
          } else if (ep.out_kind == REPQ_OUT_BF16) {
            __nv_bfloat16* o = static_cast<__nv_bfloat16*>(ep.out) + m * ep.ldo + col;
            o[0] = __float2bfloat16_rn(v[0]);
            if (two) o[1] = __float2bfloat16_rn(v[1]);
          } else if (ep.pack4) {
            static_cast<uint8_t*>(ep.out)[m * ep.ldo + (col >> 1)] = uint8_t(q[0] | (q[1] << 4));
          } else {
            uint8_t* o = static_cast<uint8_t*>(ep.out) + m * ep.ldo + col;
            o[0] = uint8_t(q[0]);
            if (two) o[1] = uint8_t(q[1]);
          }
        }
      }
      if (ep.out_row_sum != nullptr && ep.out_kind == REPQ_OUT_CODES) {
        code_sum += __shfl_xor_sync(0xffffffffu, code_sum, 1);
        code_sum += __shfl_xor_sync(0xffffffffu, code_sum, 2);
        if (t == 0 && row_ok) atomicAdd(ep.out_row_sum + m, code_sum);
      }
    }
  }
}

}  // namespace

repq_status qgemm_mma(const repq_gemm_desc& d, const EpilogueParams& ep, cudaStream_t st) {
  MmaOperand A{d.a_codes, d.lda_bytes, d.M, packed4(d.bits_a) ? 4 : 8};
  MmaOperand W{d.w_codes, d.ldw_bytes, d.N, packed4(d.bits_w) ? 4 : packed6(d.bits_w) ? 6 : 8};
  auto al = [](const uint8_t* p, int64_t ld, int64_t so, int64_t si, int bits) {
    const int64_t unit = packed4(bits) ? 2 : 4;
    return aligned(p, size_t(unit)) && ld % unit == 0 && so % unit == 0 && si % unit == 0;
  };
  const bool a_al = al(d.a_codes, d.lda_bytes, d.a_stride_outer, d.a_stride_inner, d.bits_a);
  const bool w_al = al(d.w_codes, d.ldw_bytes, d.w_stride_outer, d.w_stride_inner, d.bits_w);
  const int64_t batch = int64_t(d.batch_outer) * d.batch_inner;
  REPQ_REQUIRE(batch <= 65535, REPQ_UNSUPPORTED, "qgemm: more than 65535 batched products");
  dim3 grid((d.N + BN - 1) / BN, (d.M + BM - 1) / BM, unsigned(batch));
  REPQ_REQUIRE(grid.y <= 65535, REPQ_UNSUPPORTED, "qgemm: M too large for the warp-MMA path");
  qgemm_mma_kernel<<<grid, kThreads, 0, st>>>(A, W, d.K, d.batch_inner, d.a_stride_outer, d.a_stride_inner,
                                              d.w_stride_outer, d.w_stride_inner, d.o_stride_outer,
                                              d.o_stride_inner, a_al, w_al, ep);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace repq
