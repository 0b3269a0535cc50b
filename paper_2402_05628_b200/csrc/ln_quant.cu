// Fused LayerNorm + layer-wise uniform quantization (Eq. 9 with the reparameterized affine factors of
// Eq. 12, then Eq. 4 with the scalar (s~, z~)).
//
// HBM-bound: every input element is read once with 128-bit loads and leaves as a 4-bit (or 8-bit)
// code.  A row is owned by a group of TPR threads which keeps its slice of the row in registers, so mean
// and centred variance are two register passes with shuffle reductions.  Each group works on one or two rows
// at a time, and the rows of its next iteration are requested before the current ones are reduced, so that
// loads stay in flight all the time.
// The per-channel factors gamma~/s~ and beta~/s~ are staged once per CTA in shared memory (halves of the 8-element
// chunks apart, so that a warp's 16-byte reads are free of bank conflicts), or, for rows of 3080 to 4096 bf16 elements,
// kept in the registers of the thread that owns their columns.
//
// The float work runs on packed pairs (two elements per add / mul / fma issue slot).  Rounding is done by the
// float adder: t + 1.5 * 2^23 leaves rint(t) (half to even, on t itself, as Eq. 4 has it) in the low mantissa
// bits while |t| < 2^22; inputs that cannot guarantee that bound are clamped and converted with cvt.rni
// instead.  z is added as an integer and the clip of Eq. 4 is the saturation of the packing instruction.
#include <cuda_bf16.h>

#include "common.h"
#include "f32x2.cuh"

namespace repq {
namespace {

constexpr int kChunk = 8;   // elements per 128-bit bf16 load
constexpr int kMaxVPT = 4;  // chunks per thread: 1..4, chosen per row length

// Rows a thread group works on at a time (the loads of the next ones are always in flight as well): two,
// except where four chunks per thread would cost a resident block (measured: 16 x 3 / 32 x 3 / 256 x 4 threads x
// chunks run best with two rows, 32 x 4 / 128 x 4 with one).
__host__ __device__ constexpr int rows_in_flight(int vpt, int tpr) { return vpt >= 4 && tpr < 256 ? 1 : 2; }

// Where a thread's slice of gamma~/s~ and beta~/s~ stays in registers for the whole kernel instead of being read from
// shared memory for every pair of rows: two chunks per thread at most (32 registers) in groups of at least 128 threads,
// bf16 input (two resident blocks of 256 threads at 108 registers; measured at D = 4096: 670 -> 595 us for 262144 rows,
// three blocks with spills or one row at a time were slower).
__host__ __device__ constexpr bool factors_in_registers(int vpt, int tpr, int elem_bytes) {
  return vpt <= 2 && tpr >= 128 && elem_bytes == 2;
}

// A chunk of 8 elements as it is loaded (kept in this form while the rows before it are processed), and
// its expansion into 4 packed float pairs.
template <typename T> struct RawChunk;
template <> struct RawChunk<float> { float4 a, b; };
template <> struct RawChunk<__nv_bfloat16> { uint4 a; };

__device__ __forceinline__ void load_raw(const float* p, bool on, RawChunk<float>& r) {
  r.a = r.b = make_float4(0.f, 0.f, 0.f, 0.f);
  if (on) {
    r.a = __ldcs(reinterpret_cast<const float4*>(p));
    r.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  }
}
__device__ __forceinline__ void load_raw(const __nv_bfloat16* p, bool on, RawChunk<__nv_bfloat16>& r) {
  r.a = make_uint4(0u, 0u, 0u, 0u);
  if (on) r.a = __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ void expand(const RawChunk<float>& r, f32x2 (&v)[kChunk / 2]) {
  v[0] = pack2(r.a.x, r.a.y); v[1] = pack2(r.a.z, r.a.w); v[2] = pack2(r.b.x, r.b.y); v[3] = pack2(r.b.z, r.b.w);
}
__device__ __forceinline__ void expand(const RawChunk<__nv_bfloat16>& r, f32x2 (&v)[kChunk / 2]) {
  const uint32_t w[4] = {r.a.x, r.a.y, r.a.z, r.a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) v[i] = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
}

// Two consecutive codes (even index e0 in the low nibble) pushed into the low byte of a word that already
// holds the codes of the following pairs: d = (c << 8) | sat4(e1) << 4 | sat4(e0), saturation to [0, 15].
__device__ __forceinline__ uint32_t push_pair_u4(int e0, int e1, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.u4.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(e1), "r"(e0), "r"(c));
  return d;
}
// The same for byte codes: d = (c << 16) | sat8(e1) << 8 | sat8(e0), saturation to [0, 255].
__device__ __forceinline__ uint32_t push_pair_u8(int e0, int e1, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(e1), "r"(e0), "r"(c));
  return d;
}

// Sum over the TPR threads of a group, for kRows values at once.  Inside a warp: xor shuffles (two rows travel as one
// packed pair per add; integers take the warp-wide reduction instruction).  Across the warps of a group: lane 0 of
// every warp leaves its partial sums in shared memory, and after the barrier the first TPR / 32 lanes of every warp pick
// up one warp's partials each and finish with log2(TPR / 32) more shuffle steps (instead of every thread adding up all
// partials itself).
// Barrier of one thread group: the whole block where a group is the block, else a named barrier of the group's own (the
// groups of a block then no longer wait for one another).
template <int TPR>
__device__ __forceinline__ void group_sync(int group_first_warp) {
  if constexpr (TPR >= 256) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"r"(1 + group_first_warp / (TPR / 32)), "n"(TPR) : "memory");
}

template <int TPR, int kRows>
__device__ __forceinline__ void group_reduce(float (&v)[kRows], float* red, int group_first_warp) {
  constexpr int kShfl = TPR < 32 ? TPR : 32;
  const bool odd = threadIdx.x & 1;
  if constexpr (kRows == 2 && kShfl >= 4) {
    // neighbouring lanes split the two rows between them (one shuffle for both rows), every further step then moves one
    // value per lane, and a last exchange hands each lane the other row's total: kShfl's log + 1 shuffles instead of
    // twice the log.  All lanes of a parity add the same pairs at every step, so they end with the same bits.
    float t = (odd ? v[1] : v[0]) + __shfl_xor_sync(0xffffffffu, odd ? v[0] : v[1], 1);
#pragma unroll
    for (int o = kShfl / 2; o > 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if constexpr (TPR <= 32) {
      const float u = __shfl_xor_sync(0xffffffffu, t, 1);
      v[0] = odd ? u : t;
      v[1] = odd ? t : u;
    } else {
      v[0] = t;      // even lanes: row 0, odd lanes: row 1 (lanes 0 and 1 leave them in shared memory)
    }
  } else if constexpr (kRows == 2) {
    f32x2 p = pack2(v[0], v[1]);
#pragma unroll
    for (int o = kShfl / 2; o > 0; o >>= 1) {
      float a, b;
      unpack2(p, a, b);
      p = add2(p, pack2(__shfl_xor_sync(0xffffffffu, a, o), __shfl_xor_sync(0xffffffffu, b, o)));
    }
    unpack2(p, v[0], v[1]);
  } else {
#pragma unroll
    for (int o = kShfl / 2; o > 0; o >>= 1)
#pragma unroll
      for (int r = 0; r < kRows; ++r) v[r] += __shfl_xor_sync(0xffffffffu, v[r], o);
  }
  if constexpr (TPR > 32) {
    constexpr int kWarps = TPR / 32;
    const int lane = threadIdx.x & 31;
    if constexpr (kRows == 2) {
      // lanes 0 and 1 hold the warp's sums of rows 0 and 1.  After the barrier lane l takes row (l mod 2) of warp
      // (l / 2 mod kWarps): xor steps over the warp index, then one exchange between neighbours.
      if (lane < 2) red[(threadIdx.x >> 5) * 2 + lane] = v[0];
      group_sync<TPR>(group_first_warp);
      float t = red[(group_first_warp + ((lane >> 1) & (kWarps - 1))) * 2 + (lane & 1)];
#pragma unroll
      for (int o = kWarps; o > 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      const float u = __shfl_xor_sync(0xffffffffu, t, 1);
      v[0] = odd ? u : t;
      v[1] = odd ? t : u;
    } else {
      if (lane == 0)
#pragma unroll
        for (int r = 0; r < kRows; ++r) red[(threadIdx.x >> 5) * kRows + r] = v[r];
      group_sync<TPR>(group_first_warp);
      // lane l < kWarps takes the partials of warp l of its group; the other lanes repeat them (l mod kWarps), so that
      // the xor steps below leave the full sum in every lane
      const float* src = red + (group_first_warp + (lane & (kWarps - 1))) * kRows;
#pragma unroll
      for (int r = 0; r < kRows; ++r) v[r] = src[r];
#pragma unroll
      for (int o = kWarps / 2; o > 0; o >>= 1)
#pragma unroll
        for (int r = 0; r < kRows; ++r) v[r] += __shfl_xor_sync(0xffffffffu, v[r], o);
    }
  }
}
template <int TPR, int kRows>
__device__ __forceinline__ void group_reduce(int (&v)[kRows], int* red, int group_first_warp) {
  if constexpr (TPR >= 32) {
#pragma unroll
    for (int r = 0; r < kRows; ++r) v[r] = __reduce_add_sync(0xffffffffu, v[r]);
  } else {
#pragma unroll
    for (int o = TPR / 2; o > 0; o >>= 1)
#pragma unroll
      for (int r = 0; r < kRows; ++r) v[r] += __shfl_xor_sync(0xffffffffu, v[r], o);
  }
  if constexpr (TPR > 32) {
    constexpr int kWarps = TPR / 32;
    const int lane = threadIdx.x & 31;
    if (lane == 0)
#pragma unroll
      for (int r = 0; r < kRows; ++r) red[(threadIdx.x >> 5) * kRows + r] = v[r];
    group_sync<TPR>(group_first_warp);
    const int* src = red + (group_first_warp + (lane & (kWarps - 1))) * kRows;
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      // every group of kWarps consecutive lanes holds all partials: the warp-wide sum counts each 32 / kWarps times
      v[r] = __reduce_add_sync(0xffffffffu, src[r]) / (32 / kWarps);
    }
  }
}

template <typename T, int TPR, int kVPT, bool kPack4, bool kFull>
__global__ void __launch_bounds__((TPR > 256 ? TPR : 256),
                                  (kVPT <= 2 && TPR == 256 ? (factors_in_registers(kVPT, TPR, sizeof(T)) ? 2 : 3) : 0))
ln_quant_kernel(const T* __restrict__ x, int64_t rows, int D, int64_t ldx,
                const float* __restrict__ gamma_t, const float* __restrict__ beta_t, float eps, int rms,
                float inv_s, int z, int qmax, uint8_t* __restrict__ codes, int64_t ldc,
                int32_t* __restrict__ row_sum) {
  constexpr int kRows = rows_in_flight(kVPT, TPR);
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kGroups = kBlock / TPR;
  constexpr int kRowsPerBlock = kGroups * kRows;
  constexpr bool kRegFactors = factors_in_registers(kVPT, TPR, sizeof(T));
  extern __shared__ __align__(16) float s_gb[];          // g[D] then b[D]: gamma~/s~ and beta~/s~ (unless in registers)
  // One array per reduction of a row.  A slot may be overwritten only after every thread of the block has passed
  // a barrier that follows its reads of the slot.  With two or three reductions per iteration the barrier of the
  // next reduction is that barrier; the mean-free form without row sums has the variance reduction alone (one
  // barrier per iteration), so red_b alternates between two halves by iteration parity: the write of iteration
  // k + 2 follows the barrier of iteration k + 1, which every thread reaches after its reads of iteration k.
  __shared__ __align__(8) float red_a[kBlock / 32 * kRows];
  __shared__ __align__(8) float red_b[2][kBlock / 32 * kRows];
  __shared__ __align__(8) int red_c[kBlock / 32 * kRows];

  float* s_g = s_gb;
  float* s_b = s_gb + D;
  // |t| <= sqrt(D) |gamma~/s~| + |beta~/s~|.  While that bound stays below 2^22 the round operation is one packed
  // float add of 1.5 * 2^23 (round half to even by the adder, rint(t) left in the low mantissa bits); otherwise t
  // is clamped and converted, so that adding z cannot wrap (a whole-kernel decision, taken here once).
  const float root_d = sqrtf(float(D));
  bool wide = false;
  f32x2 g_reg[kRegFactors ? kVPT : 1][kChunk / 2], b_reg[kRegFactors ? kVPT : 1][kChunk / 2];
  if constexpr (kRegFactors) {
    // every thread works on the same columns of every row: its factors are loaded once
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int c = threadIdx.x % TPR + i * TPR;
      const bool on = kFull || c < D / kChunk;
      float gi[kChunk], bi[kChunk];
#pragma unroll
      for (int e = 0; e < kChunk; ++e) {
        gi[e] = on ? __ldg(gamma_t + c * kChunk + e) * inv_s : 0.f;
        bi[e] = on ? __ldg(beta_t + c * kChunk + e) * inv_s : 0.f;
      }
#pragma unroll
      for (int e = 0; e < kChunk; ++e) wide = wide || !(fabsf(gi[e]) * root_d + fabsf(bi[e]) < 4.0e6f);
#pragma unroll
      for (int e = 0; e < kChunk / 2; ++e) {
        g_reg[i][e] = pack2(gi[2 * e], gi[2 * e + 1]);
        b_reg[i][e] = pack2(bi[2 * e], bi[2 * e + 1]);
      }
    }
  } else {
    // layout: the first halves (4 floats) of all chunks, then the second halves, so that the 16-byte reads of
    // neighbouring lanes are neighbours in shared memory (chunk by chunk they would sit 32 bytes apart: two-way
    // bank conflicts)
    const int half_stride = D / 2;
    for (int i = threadIdx.x; i < D; i += kBlock) {
      const float gi = __ldg(gamma_t + i) * inv_s, bi = __ldg(beta_t + i) * inv_s;
      const int at = ((i >> 2) & 1) * half_stride + (i >> 3) * 4 + (i & 3);
      s_g[at] = gi;
      s_b[at] = bi;
      wide = wide || !(fabsf(gi) * root_d + fabsf(bi) < 4.0e6f);
    }
  }
  const bool guard = __syncthreads_or(wide) != 0;
  // gamma~ and beta~ are parameters; x and the outputs belong to the chain of kernels
  grid_dependency_wait();
  grid_dependency_trigger();

  const int tig = threadIdx.x % TPR;             // thread in group
  const int group = threadIdx.x / TPR;
  const int group_first_warp = (group * TPR) >> 5;
  const int nchunks = D / kChunk;
  const float inv_d = 1.f / float(D);
  const uint32_t qmax4 = uint32_t(qmax) * 0x01010101u;
  constexpr uint32_t kMagicBits = 0x4B400000u;   // 1.5 * 2^23
  const f32x2 magic2 = splat2(__uint_as_float(kMagicBits));
  const int z_less_magic = z - int(kMagicBits);

  // The rows of the next iteration are requested while those of the current one are processed, so that loads
  // stay in flight through the reductions and the packing.
  RawChunk<T> raw[kRows][kVPT];
  auto fetch = [&](int64_t first_row) {
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      // rows past the end re-read the last row (their codes are never stored); when the row fills the group
      // exactly (kFull) no load is predicated
      const int64_t row = first_row + r < rows ? first_row + r : rows - 1;
      const T* xr = x + row * ldx;
#pragma unroll
      for (int i = 0; i < kVPT; ++i) {
        const int c = tig + i * TPR;
        load_raw(xr + c * kChunk, kFull || c < nchunks, raw[r][i]);
      }
    }
  };
  const int64_t stride = int64_t(gridDim.x) * kRowsPerBlock;
  fetch(int64_t(blockIdx.x) * kRowsPerBlock + group * kRows);

  int parity = 0;
  for (int64_t base = int64_t(blockIdx.x) * kRowsPerBlock; base < rows; base += stride, parity ^= 1) {
    const int64_t row0 = base + group * kRows;

    f32x2 v[kRows][kVPT][kChunk / 2];
    float sum[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r)
#pragma unroll
      for (int i = 0; i < kVPT; ++i) expand(raw[r][i], v[r][i]);
    fetch(row0 + stride);
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      f32x2 acc = 0ull;
#pragma unroll
      for (int i = 0; i < kVPT; ++i)
#pragma unroll
        for (int e = 0; e < kChunk / 2; ++e) acc = add2(acc, v[r][i][e]);
      float lo, hi;
      unpack2(acc, lo, hi);
      sum[r] = lo + hi;
    }

    float mu[kRows];
    if (!rms) {
      group_reduce<TPR, kRows>(sum, red_a, group_first_warp);
#pragma unroll
      for (int r = 0; r < kRows; ++r) mu[r] = sum[r] * inv_d;
    } else {
#pragma unroll
      for (int r = 0; r < kRows; ++r) mu[r] = 0.f;
    }

    float ss[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const f32x2 neg_mu = splat2(-mu[r]);
      f32x2 acc = 0ull;
#pragma unroll
      for (int i = 0; i < kVPT; ++i) {
        if (kFull || tig + i * TPR < nchunks) {
#pragma unroll
          for (int e = 0; e < kChunk / 2; ++e) {
            v[r][i][e] = add2(v[r][i][e], neg_mu);
            acc = fma2(v[r][i][e], v[r][i][e], acc);
          }
        }
      }
      float lo, hi;
      unpack2(acc, lo, hi);
      ss[r] = lo + hi;
    }
    group_reduce<TPR, kRows>(ss, red_b[parity], group_first_warp);
    f32x2 rstd[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) rstd[r] = splat2(rsqrtf(ss[r] * inv_d + eps));

    int csum[kRows];
    bool live[kRows];
    uint8_t* out[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      csum[r] = 0;
      live[r] = row0 + r < rows;
      out[r] = codes + (row0 + r) * ldc;
    }
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int c = tig + i * TPR;
      if (kFull || c < nchunks) {
        f32x2 g[kChunk / 2], b[kChunk / 2];
        if constexpr (kRegFactors) {
#pragma unroll
          for (int e = 0; e < kChunk / 2; ++e) { g[e] = g_reg[i][e]; b[e] = b_reg[i][e]; }
        } else {
          const float4 g0 = *reinterpret_cast<const float4*>(s_g + c * 4);
          const float4 g1 = *reinterpret_cast<const float4*>(s_g + D / 2 + c * 4);
          const float4 b0 = *reinterpret_cast<const float4*>(s_b + c * 4);
          const float4 b1 = *reinterpret_cast<const float4*>(s_b + D / 2 + c * 4);
          g[0] = pack2(g0.x, g0.y); g[1] = pack2(g0.z, g0.w); g[2] = pack2(g1.x, g1.y); g[3] = pack2(g1.z, g1.w);
          b[0] = pack2(b0.x, b0.y); b[1] = pack2(b0.z, b0.w); b[2] = pack2(b1.x, b1.y); b[3] = pack2(b1.z, b1.w);
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
          // Eq. 4: clip(round(t) + z, 0, qmax): round half to even by the float -> int conversion, then the
          // packing instruction saturates to the container ([0, 15] or [0, 255])
          int q[kChunk];
          if (!guard) {
#pragma unroll
            for (int e = 0; e < kChunk / 2; ++e) {
              float u0, u1;
              unpack2(add2(fma2(mul2(v[r][i][e], rstd[r]), g[e], b[e]), magic2), u0, u1);
              q[2 * e] = __float_as_int(u0) + z_less_magic;
              q[2 * e + 1] = __float_as_int(u1) + z_less_magic;
            }
          } else {
            float t[kChunk];
#pragma unroll
            for (int e = 0; e < kChunk / 2; ++e) unpack2(fma2(mul2(v[r][i][e], rstd[r]), g[e], b[e]), t[2 * e], t[2 * e + 1]);
#pragma unroll
            for (int e = 0; e < kChunk; ++e) q[e] = __float2int_rn(fminf(fmaxf(t[e], -1.0e9f), 1.0e9f)) + z;
          }
          // rows past the end compute on a copy of the last row; only the stores are predicated
          if constexpr (kPack4) {
            uint32_t w = 0;
#pragma unroll
            for (int e = kChunk - 2; e >= 0; e -= 2) w = push_pair_u4(q[e], q[e + 1], w);
            if (live[r]) reinterpret_cast<uint32_t*>(out[r])[c] = w;
            csum[r] = int(__dp4a(w & 0x0F0F0F0Fu, 0x01010101u, __dp4a((w >> 4) & 0x0F0F0F0Fu, 0x01010101u, uint32_t(csum[r]))));
          } else {
            uint2 w;
            w.x = push_pair_u8(q[0], q[1], push_pair_u8(q[2], q[3], 0u));
            w.y = push_pair_u8(q[4], q[5], push_pair_u8(q[6], q[7], 0u));
            w.x = __vminu4(w.x, qmax4);          // 4- and 6-bit quantizers in byte containers
            w.y = __vminu4(w.y, qmax4);
            if (live[r]) reinterpret_cast<uint2*>(out[r])[c] = w;
            csum[r] = int(__dp4a(w.x, 0x01010101u, __dp4a(w.y, 0x01010101u, uint32_t(csum[r]))));
          }
        }
      }
    }
    if (row_sum != nullptr) {
      group_reduce<TPR, kRows>(csum, red_c, group_first_warp);
      if (tig == 0) {
#pragma unroll
        for (int r = 0; r < kRows; ++r)
          if (row0 + r < rows) row_sum[row0 + r] = csum[r];
      }
    }
  }
}

template <typename T, int TPR, int kVPT>
repq_status launch(const T* x, int64_t rows, int D, int64_t ldx, const float* g, const float* b, float eps,
                   int rms, float s_t, int z, int bits, uint8_t* codes, int64_t ldc, int32_t* row_sum,
                   cudaStream_t st) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR * rows_in_flight(kVPT, TPR);
  const int64_t need = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
  const float inv_s = 1.f / s_t;
  const int qmax = code_max(bits);
  const size_t smem = factors_in_registers(kVPT, TPR, sizeof(T)) ? 0 : size_t(D) * 2 * sizeof(float);
  const bool full = D == TPR * kVPT * kChunk;   // the row fills the group exactly: no chunk is predicated
  auto kern = packed4(bits) ? (full ? ln_quant_kernel<T, TPR, kVPT, true, true> : ln_quant_kernel<T, TPR, kVPT, true, false>)
                            : (full ? ln_quant_kernel<T, TPR, kVPT, false, true> : ln_quant_kernel<T, TPR, kVPT, false, false>);
  if (smem > 48 * 1024) REPQ_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  // persistent grid: exactly the blocks that are resident at once, so that every block keeps its load pipeline
  // running over all of its rows
  int resident = 0;
  REPQ_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kern, kBlock, smem));
  const int64_t cap = int64_t(sm_count()) * (resident > 0 ? resident : 1);
  const int grid = int(need < cap ? need : cap);
  REPQ_CUDA(launch_chained(kern, dim3(grid), dim3(kBlock), smem, st, x, rows, D, ldx, g, b, eps, rms, inv_s, z, qmax, codes, ldc, row_sum));
  note_launch();
  return REPQ_OK;
}

template <typename T, int TPR>
repq_status launch_vpt(int vpt, const T* x, int64_t rows, int D, int64_t ldx, const float* g, const float* b, float eps,
                       int rms, float s_t, int z, int bits, uint8_t* codes, int64_t ldc, int32_t* row_sum,
                       cudaStream_t st) {
  switch (vpt) {
    case 1: return launch<T, TPR, 1>(x, rows, D, ldx, g, b, eps, rms, s_t, z, bits, codes, ldc, row_sum, st);
    case 2: return launch<T, TPR, 2>(x, rows, D, ldx, g, b, eps, rms, s_t, z, bits, codes, ldc, row_sum, st);
    case 3: return launch<T, TPR, 3>(x, rows, D, ldx, g, b, eps, rms, s_t, z, bits, codes, ldc, row_sum, st);
    default: return launch<T, TPR, 4>(x, rows, D, ldx, g, b, eps, rms, s_t, z, bits, codes, ldc, row_sum, st);
  }
}

template <typename T>
repq_status dispatch(const T* x, int64_t rows, int D, int64_t ldx, const float* g, const float* b, float eps,
                     int rms, float s_t, int z, int bits, uint8_t* codes, int64_t ldc, int32_t* row_sum,
                     cudaStream_t st) {
  const int nchunks = D / kChunk;
  // a row that would take four chunks per thread in a group of 128 goes to a whole block with two (measured:
  // D = 4096 runs 9 % faster as 256 x 2 with three resident blocks than as 128 x 4 with one)
#define REPQ_LN_CASE(TPR) \
  if (nchunks <= TPR * (TPR == 128 ? 3 : kMaxVPT)) return launch_vpt<T, TPR>((nchunks + TPR - 1) / TPR, x, rows, D, ldx, g, b, eps, rms, s_t, z, bits, codes, ldc, row_sum, st);
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
