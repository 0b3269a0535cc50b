// Fused Softmax -> log2-domain codes of the log-sqrt2 quantizer (Eq. 3's Softmax, then Eq. 15).
//
// With m = max_j S_j and Z = sum_j 2^(c (S_j - m)), c = pre_scale * log2(e), the value handed to the
// round operation of Eq. 15 is
//     -2 log2(A_i / s) = 2 (log2 Z + log2 s) - 2 c (S_i - m),
// so the probabilities themselves are never formed: one exp2 per element for Z, one FMA per element
// for the code, and no underflow (a key whose probability would underflow simply lands on the top
// code, as the clip in Eq. 15 demands).
//
// HBM-bound: each score is read once (128-bit loads, row kept in registers by a group of TPR threads)
// and leaves as a 4-bit or 8-bit code.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "common.h"
#include "f32x2.cuh"

namespace repq {
namespace {

constexpr int kChunk = 8;
constexpr int kMaxVPT = 4;   // chunks per thread: 1..4, chosen per row length
constexpr uint32_t kMagicBits = 0x4B400000u;   // 1.5 * 2^23

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Elements [idx, idx + 8) of a row.  Fast form: the whole chunk is visible and one or two 128-bit loads cover
// it; it is requested one row ahead, kept as loaded, and expanded into 4 packed pairs when its row's turn comes.
template <typename T> struct RawChunk;
template <> struct RawChunk<float> { float4 a, b; };
template <> struct RawChunk<__nv_bfloat16> { uint4 a; };
__device__ __forceinline__ void load_raw(const float* p, RawChunk<float>& r) {
  r.a = __ldcs(reinterpret_cast<const float4*>(p));
  r.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
}
__device__ __forceinline__ void load_raw(const __nv_bfloat16* p, RawChunk<__nv_bfloat16>& r) {
  r.a = __ldcs(reinterpret_cast<const uint4*>(p));
}
// The same with the second 16 bytes of a float chunk optional (a row stride that ends inside the last chunk).
__device__ __forceinline__ void load_raw_part(const float* p, bool second, RawChunk<float>& r) {
  r.a = __ldcs(reinterpret_cast<const float4*>(p));
  if (second) r.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
}
__device__ __forceinline__ void load_raw_part(const __nv_bfloat16* p, bool, RawChunk<__nv_bfloat16>& r) {
  r.a = __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ void expand(const RawChunk<float>& r, f32x2 (&v)[kChunk / 2]) {
  v[0] = pack2(r.a.x, r.a.y); v[1] = pack2(r.a.z, r.a.w); v[2] = pack2(r.b.x, r.b.y); v[3] = pack2(r.b.z, r.b.w);
}
__device__ __forceinline__ void expand(const RawChunk<__nv_bfloat16>& r, f32x2 (&v)[kChunk / 2]) {
  const uint32_t w[4] = {r.a.x, r.a.y, r.a.z, r.a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) v[i] = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
}
// General form (kept out of line: it runs for rows that are not 16-byte aligned and for a chunk that would
// cross the row stride): element loads, -inf at or beyond `valid`.
struct ChunkPairs { f32x2 p0, p1, p2, p3; };
__device__ __noinline__ ChunkPairs load_ragged(const float* row, int idx, int valid) {
  float f[kChunk];
  for (int e = 0; e < kChunk; ++e) f[e] = (idx + e < valid) ? __ldcs(row + idx + e) : -CUDART_INF_F;
  return ChunkPairs{pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7])};
}
__device__ __noinline__ ChunkPairs load_ragged(const __nv_bfloat16* row, int idx, int valid) {
  float f[kChunk];
  for (int e = 0; e < kChunk; ++e) f[e] = (idx + e < valid) ? __bfloat162float(row[idx + e]) : -CUDART_INF_F;
  return ChunkPairs{pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7])};
}

// Two consecutive codes (even index first) pushed into the low byte / low half of a word that already holds the
// codes after them, with saturation to [0, 15] / [0, 255] (cvt.pack.sat: d = c << 8 | sat(e1) << 4 | sat(e0)).
__device__ __forceinline__ uint32_t push_pair_u4(int e0, int e1, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.u4.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(e1), "r"(e0), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t push_pair_u8(int e0, int e1, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(e1), "r"(e0), "r"(c));
  return d;
}

template <int TPR, bool kMax>
__device__ __forceinline__ float group_reduce(float v, float* red, int group_first_warp) {
  constexpr int kShfl = TPR < 32 ? TPR : 32;
#pragma unroll
  for (int o = kShfl / 2; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, v, o);
    v = kMax ? fmaxf(v, other) : v + other;
  }
  if constexpr (TPR > 32) {
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    v = kMax ? -CUDART_INF_F : 0.f;
#pragma unroll
    for (int w = 0; w < TPR / 32; ++w) {
      const float other = red[group_first_warp + w];
      v = kMax ? fmaxf(v, other) : v + other;
    }
  }
  return v;
}

template <typename T, int TPR, int kVPT, bool kPack4>
__global__ void __launch_bounds__((TPR > 256 ? TPR : 256))
softmax_log2_kernel(const T* __restrict__ scores, int64_t rows, int L, int64_t ld, bool vec_ok, float c,
                    int causal_period, int causal_offset, float log2_s, int qmax,
                    uint8_t* __restrict__ codes, int64_t ldc) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR;
  __shared__ float red_a[kBlock / 32];
  __shared__ float red_b[kBlock / 32];

  const int tig = threadIdx.x % TPR;
  const int group = threadIdx.x / TPR;
  const int group_first_warp = (group * TPR) >> 5;
  const int nchunks = (L + kChunk - 1) / kChunk;
  const float fq = float(qmax);

  // keys a row may see (0 for rows past the end)
  auto visible = [&](int64_t row) {
    if (row >= rows) return 0;
    if (causal_period <= 0) return L;
    const int64_t v = (row % causal_period) + 1 + causal_offset;
    return v < 1 ? 1 : (v < L ? int(v) : L);
  };
  // The vector-loadable chunks (16-byte aligned rows, chunk inside the row stride) of the next row of this group are requested while the current row
  // is processed, so that loads stay in flight through the reductions.
  RawChunk<T> raw[kVPT];
  auto fetch = [&](int64_t row) {
    const int valid = visible(row);
    const T* sr = scores + (row < rows ? row : 0) * ld;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int idx = (tig + i * TPR) * kChunk;
      if (vec_ok && idx < valid && idx + kChunk <= ld) load_raw(sr + idx, raw[i]);
    }
  };
  const int64_t stride = int64_t(gridDim.x) * kRowsPerBlock;
  fetch(int64_t(blockIdx.x) * kRowsPerBlock + group);

  for (int64_t base = int64_t(blockIdx.x) * kRowsPerBlock; base < rows; base += stride) {
    const int64_t row = base + group;
    const bool live = row < rows;
    const T* sr = scores + (live ? row : 0) * ld;
    const int valid = visible(row);

    // the row slice of this thread as packed pairs; masked keys (at or beyond `valid`) are -inf
    f32x2 v[kVPT][kChunk / 2];
    float m = -CUDART_INF_F;
    const f32x2 ninf2 = splat2(-CUDART_INF_F);
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int ch = tig + i * TPR;
      const int idx = ch * kChunk;
      if (idx >= valid) {                                    // (also: chunks past the row, rows past the end)
#pragma unroll
        for (int e = 0; e < kChunk / 2; ++e) v[i][e] = ninf2;
        continue;
      }
      if (vec_ok && idx + kChunk <= ld) {
        expand(raw[i], v[i]);
        if (idx + kChunk > valid) {                          // the chunk that holds the row's last visible key
#pragma unroll
          for (int e = 0; e < kChunk / 2; ++e) {
            float lo, hi;
            unpack2(v[i][e], lo, hi);
            v[i][e] = pack2(idx + 2 * e < valid ? lo : -CUDART_INF_F, idx + 2 * e + 1 < valid ? hi : -CUDART_INF_F);
          }
        }
      } else {
        const ChunkPairs r = load_ragged(sr, idx, valid);
        v[i][0] = r.p0; v[i][1] = r.p1; v[i][2] = r.p2; v[i][3] = r.p3;
      }
#pragma unroll
      for (int e = 0; e < kChunk / 2; ++e) {
        float lo, hi;
        unpack2(v[i][e], lo, hi);
        m = fmaxf(m, fmaxf(lo, hi));
      }
    }
    fetch(row + stride);
    m = group_reduce<TPR, true>(m, red_a, group_first_warp);
    if (!live) m = 0.f;

    // d = S - m (<= 0, -inf for masked keys); Z = sum 2^(c d)
    const f32x2 neg_m = splat2(-m), c2 = splat2(c);
    float z = 0.f;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      if ((tig + i * TPR) * kChunk >= valid) continue;          // chunk fully masked: contributes nothing
#pragma unroll
      for (int e = 0; e < kChunk / 2; ++e) {
        v[i][e] = add2(v[i][e], neg_m);
        float a0, a1;
        unpack2(mul2(v[i][e], c2), a0, a1);
        z += ex2(a0) + ex2(a1);
      }
    }
    z = group_reduce<TPR, false>(z, red_b, group_first_warp);
    const f32x2 k0 = splat2(2.f * (log2f(z) + log2_s));
    const f32x2 k1 = splat2(-2.f * c);
    const f32x2 magic2 = splat2(__uint_as_float(kMagicBits));

    if (live) {
      uint8_t* out = codes + row * ldc;
#pragma unroll
      for (int i = 0; i < kVPT; ++i) {
        const int ch = tig + i * TPR;
        if (ch < nchunks && ch * kChunk >= valid) {
          // fully masked chunk: top codes, no arithmetic
          const uint32_t top = uint32_t(qmax) * (kPack4 ? 0x11111111u : 0x01010101u);
          if constexpr (kPack4) reinterpret_cast<uint32_t*>(out)[ch] = top;
          else reinterpret_cast<uint2*>(out)[ch] = make_uint2(top, top);
        } else if (ch < nchunks) {
          // Eq. 15: clip(round(t), 0, qmax).  The upper clip is a float min (t = +inf for masked keys and
          // underflowed probabilities lands on the top code); rounding half to even is one packed float add of
          // 1.5 * 2^23, which leaves the code in the low mantissa bits; negative t (possible for s < 1 only) would
          // leave a negative integer there, which the saturating pack turns into code 0.
          int q[kChunk];
#pragma unroll
          for (int e = 0; e < kChunk / 2; ++e) {
            float t0, t1;
            unpack2(fma2(v[i][e], k1, k0), t0, t1);
            float r0, r1;
            unpack2(add2(pack2(fminf(t0, fq), fminf(t1, fq)), magic2), r0, r1);
            q[2 * e] = __float_as_int(r0) - int(kMagicBits);
            q[2 * e + 1] = __float_as_int(r1) - int(kMagicBits);
          }
          if constexpr (kPack4) {
            uint32_t w = 0;
#pragma unroll
            for (int e = kChunk - 2; e >= 0; e -= 2) w = push_pair_u4(q[e], q[e + 1], w);
            reinterpret_cast<uint32_t*>(out)[ch] = w;
          } else {
            uint2 w;
            w.x = push_pair_u8(q[0], q[1], push_pair_u8(q[2], q[3], 0u));
            w.y = push_pair_u8(q[4], q[5], push_pair_u8(q[6], q[7], 0u));
            reinterpret_cast<uint2*>(out)[ch] = w;
          }
        }
      }
    }
  }
}

// The same computation for the common case: no causal mask, 16-byte aligned rows, and a row stride that covers
// the last chunk of 8 (or, for float32 scores, its first half when the row ends there).  Which of a thread's chunks are whole, partial or past the row is then the same for every
// row, so it is decided once; chunk slots that are whole for every thread of a group run without predicates, rows
// past the end re-read the last row (nothing of them is stored), and the upper clip of Eq. 15 is left to the
// saturating pack (t = +inf or beyond 2^22 leaves a large positive integer after the magic-number subtraction).
// kWhole: the number of whole chunk slots when it is kVPT or kVPT - 1 (known at compile time, so that those slots
// carry no test at all), -1 otherwise (taken from L at run time).
template <typename T, int TPR, int kVPT, bool kPack4, int kWhole>
__global__ void __launch_bounds__((TPR > 256 ? TPR : 256), (TPR <= 32 ? 3 : 0))
softmax_log2_plain_kernel(const T* __restrict__ scores, int64_t rows, int L, int64_t ld, bool tail_half, float c,
                          float log2_s, int qmax, uint8_t* __restrict__ codes, int64_t ldc) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR;
  __shared__ float red_a[kBlock / 32];
  __shared__ float red_b[kBlock / 32];

  const int tig = threadIdx.x % TPR;
  const int group = threadIdx.x / TPR;
  const int group_first_warp = (group * TPR) >> 5;
  const int n_full = kWhole >= 0 ? kWhole : (L / kChunk) / TPR;   // chunk slots below this are whole for every thread of a group
  int cnt[kVPT];                                // visible elements of this thread's chunk i (0..8), any row
#pragma unroll
  for (int i = 0; i < kVPT; ++i) {
    const int left = L - (tig + i * TPR) * kChunk;
    cnt[i] = left < 0 ? 0 : (left > kChunk ? kChunk : left);
  }
  const uint32_t qmax4 = uint32_t(qmax) * 0x01010101u;

  RawChunk<T> raw[kVPT];
#pragma unroll
  for (int i = 0; i < kVPT; ++i) raw[i] = RawChunk<T>{};
  auto fetch = [&](int64_t row) {
    const T* sr = scores + (row < rows ? row : rows - 1) * ld;
#pragma unroll
    for (int i = 0; i < kVPT; ++i)
      if (i < n_full || cnt[i] > 0)   // tail_half: the row's last chunk holds at most 4 keys and the stride ends after them
        load_raw_part(sr + (tig + i * TPR) * kChunk, i < n_full || !tail_half || cnt[i] > 4, raw[i]);
  };
  const int64_t stride = int64_t(gridDim.x) * kRowsPerBlock;
  fetch(int64_t(blockIdx.x) * kRowsPerBlock + group);

  const f32x2 c2 = splat2(c);
  const f32x2 k1 = splat2(-2.f * c);
  const f32x2 magic2 = splat2(__uint_as_float(kMagicBits));
  for (int64_t base = int64_t(blockIdx.x) * kRowsPerBlock; base < rows; base += stride) {
    const int64_t row = base + group;
    const bool live = row < rows;

    f32x2 v[kVPT][kChunk / 2];
    float m = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      expand(raw[i], v[i]);
      if (i >= n_full) {                         // a slot that holds the row's ragged end for some thread
#pragma unroll
        for (int e = 0; e < kChunk / 2; ++e) {
          float lo, hi;
          unpack2(v[i][e], lo, hi);
          v[i][e] = pack2(2 * e < cnt[i] ? lo : -CUDART_INF_F, 2 * e + 1 < cnt[i] ? hi : -CUDART_INF_F);
        }
      }
#pragma unroll
      for (int e = 0; e < kChunk / 2; ++e) {
        float lo, hi;
        unpack2(v[i][e], lo, hi);
        m = fmaxf(m, fmaxf(lo, hi));
      }
    }
    fetch(row + stride);
    m = group_reduce<TPR, true>(m, red_a, group_first_warp);

    // d = S - m (<= 0, -inf for keys past the row); Z = sum 2^(c d)
    const f32x2 neg_m = splat2(-m);
    f32x2 zz = 0ull;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      if (i < n_full || cnt[i] > 0) {
#pragma unroll
        for (int e = 0; e < kChunk / 2; ++e) {
          v[i][e] = add2(v[i][e], neg_m);
          float a0, a1;
          unpack2(mul2(v[i][e], c2), a0, a1);
          zz = add2(zz, pack2(ex2(a0), ex2(a1)));
        }
      }
    }
    float z0, z1;
    unpack2(zz, z0, z1);
    const float z = group_reduce<TPR, false>(z0 + z1, red_b, group_first_warp);
    const f32x2 k0 = splat2(2.f * (log2f(z) + log2_s));

    uint8_t* out = codes + row * ldc;
#pragma unroll
    for (int i = 0; i < kVPT; ++i) {
      const int ch = tig + i * TPR;
      if (i < n_full || cnt[i] > 0) {
        // Eq. 15: clip(round(t), 0, qmax); rounding half to even is one packed float add of 1.5 * 2^23, which
        // leaves the code in the low mantissa bits; both clips are the saturation of the pack (negative t,
        // possible for s < 1 only, leaves a negative integer; t = +inf for keys past the row and underflowed
        // probabilities leaves a large positive one)
        int q[kChunk];
#pragma unroll
        for (int e = 0; e < kChunk / 2; ++e) {
          float r0, r1;
          unpack2(add2(fma2(v[i][e], k1, k0), magic2), r0, r1);
          q[2 * e] = __float_as_int(r0) - int(kMagicBits);
          q[2 * e + 1] = __float_as_int(r1) - int(kMagicBits);
        }
        if constexpr (kPack4) {
          uint32_t w = 0;
#pragma unroll
          for (int e = kChunk - 2; e >= 0; e -= 2) w = push_pair_u4(q[e], q[e + 1], w);
          if (live) reinterpret_cast<uint32_t*>(out)[ch] = w;
        } else {
          uint2 w;
          w.x = __vminu4(push_pair_u8(q[0], q[1], push_pair_u8(q[2], q[3], 0u)), qmax4);   // 6-bit codes in bytes
          w.y = __vminu4(push_pair_u8(q[4], q[5], push_pair_u8(q[6], q[7], 0u)), qmax4);
          if (live) reinterpret_cast<uint2*>(out)[ch] = w;
        }
      }
    }
  }
}

template <typename T, int TPR, int kVPT>
repq_status launch(const T* scores, int64_t rows, int L, int64_t ld, bool vec_ok, float c, int period,
                   int offset, float log2_s, int bits, uint8_t* codes, int64_t ldc, cudaStream_t st) {
  constexpr int kBlock = TPR > 256 ? TPR : 256;
  constexpr int kRowsPerBlock = kBlock / TPR;
  const int64_t need = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
  const int qmax = code_max(bits);
  const int64_t chunks8 = (int64_t(L) + kChunk - 1) / kChunk * kChunk;
  const bool tail_half = chunks8 > ld && sizeof(T) == 4 && L % kChunk >= 1 && L % kChunk <= 4 && chunks8 - 4 <= ld;
  if (vec_ok && period <= 0 && (chunks8 <= ld || tail_half)) {
    const int whole = (L / kChunk) / TPR;
    auto plain = packed4(bits) ? softmax_log2_plain_kernel<T, TPR, kVPT, true, -1> : softmax_log2_plain_kernel<T, TPR, kVPT, false, -1>;
    if constexpr (TPR <= 64) {     // (measured: the compile-time count gains 2-5 % on short rows and loses 4 % with 256 threads per row)
      if (whole == kVPT) plain = packed4(bits) ? softmax_log2_plain_kernel<T, TPR, kVPT, true, kVPT> : softmax_log2_plain_kernel<T, TPR, kVPT, false, kVPT>;
      if (whole == kVPT - 1) plain = packed4(bits) ? softmax_log2_plain_kernel<T, TPR, kVPT, true, kVPT - 1> : softmax_log2_plain_kernel<T, TPR, kVPT, false, kVPT - 1>;
    }
    int fit = 0;
    REPQ_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, plain, kBlock, 0));
    const int64_t most = int64_t(sm_count()) * (fit > 0 ? fit : 1);
    plain<<<int(need < most ? need : most), kBlock, 0, st>>>(scores, rows, L, ld, tail_half, c, log2_s, qmax, codes, ldc);
    REPQ_CUDA(cudaGetLastError());
    note_launch();
    return REPQ_OK;
  }
  auto kern = packed4(bits) ? softmax_log2_kernel<T, TPR, kVPT, true> : softmax_log2_kernel<T, TPR, kVPT, false>;
  // persistent grid: exactly the blocks that are resident at once (every block keeps its load pipeline running)
  int resident = 0;
  REPQ_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kern, kBlock, 0));
  const int64_t cap = int64_t(sm_count()) * (resident > 0 ? resident : 1);
  const int grid = int(need < cap ? need : cap);
  kern<<<grid, kBlock, 0, st>>>(scores, rows, L, ld, vec_ok, c, period, offset, log2_s, qmax, codes, ldc);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

template <typename T, int TPR>
repq_status launch_vpt(int vpt, const T* scores, int64_t rows, int L, int64_t ld, bool vec_ok, float c, int period,
                       int offset, float log2_s, int bits, uint8_t* codes, int64_t ldc, cudaStream_t st) {
  switch (vpt) {
    case 1: return launch<T, TPR, 1>(scores, rows, L, ld, vec_ok, c, period, offset, log2_s, bits, codes, ldc, st);
    case 2: return launch<T, TPR, 2>(scores, rows, L, ld, vec_ok, c, period, offset, log2_s, bits, codes, ldc, st);
    case 3: return launch<T, TPR, 3>(scores, rows, L, ld, vec_ok, c, period, offset, log2_s, bits, codes, ldc, st);
    default: return launch<T, TPR, 4>(scores, rows, L, ld, vec_ok, c, period, offset, log2_s, bits, codes, ldc, st);
  }
}

template <typename T>
repq_status dispatch(const T* scores, int64_t rows, int L, int64_t ld, bool vec_ok, float c, int period,
                     int offset, float log2_s, int bits, uint8_t* codes, int64_t ldc, cudaStream_t st) {
  const int nchunks = (L + kChunk - 1) / kChunk;
#define REPQ_SM_CASE(TPR) \
  if (nchunks <= TPR * kMaxVPT) return launch_vpt<T, TPR>((nchunks + TPR - 1) / TPR, scores, rows, L, ld, vec_ok, c, period, offset, log2_s, bits, codes, ldc, st);
  REPQ_SM_CASE(8)
  REPQ_SM_CASE(16)
  REPQ_SM_CASE(32)
  REPQ_SM_CASE(64)
  REPQ_SM_CASE(128)
  REPQ_SM_CASE(256)
  REPQ_SM_CASE(512)
#undef REPQ_SM_CASE
  return fail(REPQ_UNSUPPORTED, "softmax_log2: L = %d exceeds 16384", L);
}

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_softmax_log2(const void* scores, int dtype, int64_t rows, int L, int64_t ld,
                                         float pre_scale, int causal_period, int causal_offset, float s,
                                         int bits, uint8_t* codes, int64_t ld_codes_bytes, void* stream) {
  REPQ_REQUIRE(rows >= 0 && L > 0, REPQ_INVALID_ARG, "softmax_log2: rows must be >= 0 and L > 0");
  if (rows == 0) return REPQ_OK;
  REPQ_REQUIRE(scores && codes, REPQ_INVALID_ARG, "softmax_log2: NULL pointer");
  REPQ_REQUIRE(dtype == REPQ_F32 || dtype == REPQ_BF16, REPQ_INVALID_ARG, "softmax_log2: dtype must be REPQ_F32 or REPQ_BF16");
  REPQ_REQUIRE(bits_ok(bits), REPQ_INVALID_ARG, "softmax_log2: bits must be 4, 6 or 8");
  REPQ_REQUIRE(s > 0.f && pre_scale > 0.f, REPQ_INVALID_ARG, "softmax_log2: s and pre_scale must be positive");
  REPQ_REQUIRE(ld >= L, REPQ_INVALID_ARG, "softmax_log2: ld < L");
  REPQ_REQUIRE(causal_period >= 0, REPQ_INVALID_ARG, "softmax_log2: causal_period must be >= 0");
  REPQ_REQUIRE(L <= 16384, REPQ_UNSUPPORTED, "softmax_log2: L = %d exceeds 16384", L);
  const int64_t unit = packed4(bits) ? 4 : 8;
  const int64_t need = (int64_t(L) + 7) / 8 * unit;
  REPQ_REQUIRE(ld_codes_bytes >= need, REPQ_INVALID_ARG,
               "softmax_log2: ld_codes_bytes = %lld, need at least %lld (rows are written in groups of 8 codes)",
               (long long)ld_codes_bytes, (long long)need);
  REPQ_REQUIRE(aligned(codes, unit) && ld_codes_bytes % unit == 0, REPQ_ALIGNMENT,
               "softmax_log2: codes rows must be %d-byte aligned", int(unit));
  const size_t esz = dtype == REPQ_F32 ? 4 : 2;
  REPQ_REQUIRE(aligned(scores, esz), REPQ_ALIGNMENT, "softmax_log2: scores pointer is not element-aligned");
  const bool vec_ok = aligned(scores, 16) && (size_t(ld) * esz) % 16 == 0;
  const float c = pre_scale * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == REPQ_F32)
    return dispatch(static_cast<const float*>(scores), rows, L, ld, vec_ok, c, causal_period, causal_offset, log2f(s), bits, codes, ld_codes_bytes, st);
  return dispatch(static_cast<const __nv_bfloat16*>(scores), rows, L, ld, vec_ok, c, causal_period, causal_offset, log2f(s), bits, codes, ld_codes_bytes, st);
}
