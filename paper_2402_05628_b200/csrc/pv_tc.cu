// P.V with log2-domain Softmax codes (Eqs. 16-17) on the 5th-generation tensor cores.
//
//     A^[i, j] = s 2^(-ceil(p/2)) (sqrt2 if p odd else 1),     O = A^ . (s_v (V - z_v))
//
// Even and odd codes go to two operand tiles E and O of exact bf16 powers of two (zero where the parity does
// not match), V becomes the exact bf16 integers v - z_v, and two tcgen05.mma (kind::f16, bf16 x bf16 -> f32)
// per 16 keys accumulate E.V and O.V in tensor memory.  The irrational factor of Eq. 17 is applied once, in
// float32, when the accumulators are read back:  O = s s_v (acc_E + sqrt2 acc_O).
//
// One CTA owns 128 query rows of one (batch, head) pair and walks the keys in chunks of 64:
//   warps 0..7          fetch the chunk's codes (8 lanes cover the 64 codes of a row, one chunk ahead, into
//                       registers) and expand them through a 256-entry table (a whole byte = two codes at a time
//                       for 4-bit codes) into the K-major, 128-byte-swizzled E and O tiles; convert the chunk's
//                       V rows (also fetched one chunk ahead) into a [key][channel] tile, which the MMA reads as
//                       an MN-major operand; keys past the row's limit (Lk, causal mask) are zeroed
//   warp 8 (one lane)   tensor-memory allocation and MMA issue; tcgen05.commit hands the stage back
//   warps 0..3          epilogue: one output row per thread, tcgen05.ld of both accumulators, scale,
//                       re-quantization (Eq. 4) or float output, vector stores
// Every mbarrier wait is bounded; when one runs out the kernel records a status code, all roles leave their
// loops, MMAs in flight are drained, tensor memory is freed and the kernel returns.
#include <cuda_bf16.h>

#include <cstdlib>

#include "kernels.h"
#include "tc_ptx.cuh"

namespace repq {
namespace {

using namespace tc;

constexpr int kRows = 128;                  // query rows per CTA (MMA M)
constexpr int kKeys = 64;                   // keys per chunk: one 128-byte swizzle row of bf16
constexpr int kExpWarps = 8;
constexpr int kExpThreads = 32 * kExpWarps;
constexpr int kThreads = kExpThreads + 32;
constexpr uint32_t kTileBytes = kRows * 128;      // E or O tile of one chunk
constexpr uint32_t kVBlockBytes = kKeys * 128;    // 64 keys x 64 channels of bf16
constexpr uint32_t kMagic = 0x4B400000u;          // float 1.5 * 2^23: low mantissa bits hold a small integer

template <bool kP4, int NB>
struct PvShared {
  static constexpr int kStages = 2;
  static constexpr int kCodeBox = kP4 ? 32 : 64;    // bytes of one row's 64 codes
  alignas(1024) uint8_t e[kStages][kTileBytes];
  alignas(1024) uint8_t o[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][NB * kVBlockBytes];
  alignas(16) uint32_t lut[kP4 ? 512 : 256];
  alignas(8) uint64_t ops_full[kStages];
  uint64_t ops_empty[kStages];
  uint64_t acc_full;
  uint64_t done;
  uint32_t tmem_base;
  volatile int abort;
};

struct PvTcParams {
  PvParams p;
  int n_pad;          // d_h rounded up to 16: MMA N, and the column offset of the odd accumulator
  int tmem_cols;      // power of two >= 2 n_pad, >= 32
  int vec_store;      // output rows allow 16-byte stores
  int32_t* status;
};

// bf16 bit pattern of 2^(-ceil(c/2)); zero once the exponent leaves the normal range.
__device__ __forceinline__ uint32_t pow2_bits(uint32_t c) {
  const uint32_t e = (c + 1u) >> 1;
  return e <= 126u ? (127u - e) << 7 : 0u;
}

__device__ __forceinline__ uint32_t tile_offset(int row, int chunk16) {
  return uint32_t(row >> 3) * 1024u + uint32_t(row & 7) * 128u + (uint32_t(chunk16 ^ (row & 7)) << 4);
}

// Keeps the first `limit` (0..8) bf16 elements of a 16-byte group.
__device__ __forceinline__ void keep_first(uint4& x, int limit) {
  uint32_t* w = reinterpret_cast<uint32_t*>(&x);
#pragma unroll
  for (int i = 0; i < 4; ++i)
    w[i] &= (2 * i < limit ? 0x0000FFFFu : 0u) | (2 * i + 1 < limit ? 0xFFFF0000u : 0u);
}

template <bool kP4, int NB>
__global__ void __launch_bounds__(kThreads)
pv_tc_kernel(PvTcParams T) {
  using Shared = PvShared<kP4, NB>;
  constexpr int kStages = Shared::kStages;
  constexpr int kCodeBox = Shared::kCodeBox;
  constexpr int kVItems = 2 * NB;                         // 8-channel groups of V per thread and chunk
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Shared& S = *reinterpret_cast<Shared*>(smem_raw);
  const PvParams& P = T.p;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int pair = blockIdx.y;
  const int bo = pair / P.batch_inner, bi = pair % P.batch_inner;
  const int q0 = blockIdx.x * kRows;
  const int shift = P.Lk - P.Lq;
  // keys this CTA has to visit, and the fewest keys any of its rows may attend to
  const int k_end = P.causal ? max(1, min(P.Lk, min(q0 + kRows, P.Lq) + shift)) : P.Lk;
  const int min_valid = P.causal ? max(0, min(P.Lk, q0 + 1 + shift)) : P.Lk;
  const int n_chunks = (k_end + kKeys - 1) / kKeys;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&S.ops_full[s]), kExpWarps);
      mbar_init(smem_u32(&S.ops_empty[s]), 1);
    }
    mbar_init(smem_u32(&S.acc_full), 1);
    mbar_init(smem_u32(&S.done), 1);
    S.abort = 0;
    if (smem_u32(smem_raw) & 1023u) {                      // the swizzled tiles need this alignment
      atomicCAS(T.status, 0, 29);
      S.abort = 1;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // code -> operand table: 4-bit: entry [byte] = (bf16 pair for E, bf16 pair for O) of the byte's two codes;
  // byte codes: entry [code] = E value in the low half, O value in the high half
  if (tid < 256) {
    const uint32_t i = uint32_t(tid);
    if (kP4) {
      const uint32_t c0 = i & 15u, c1 = i >> 4, b0 = pow2_bits(c0), b1 = pow2_bits(c1);
      S.lut[2 * i] = ((c0 & 1u) ? 0u : b0) | (((c1 & 1u) ? 0u : b1) << 16);
      S.lut[2 * i + 1] = ((c0 & 1u) ? b0 : 0u) | (((c1 & 1u) ? b1 : 0u) << 16);
    } else {
      const uint32_t b = pow2_bits(i);
      S.lut[i] = (i & 1u) ? (b << 16) : b;
    }
  }
  if (warp == kExpWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&S.tmem_base)), "r"(uint32_t(T.tmem_cols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S.tmem_base;
  volatile int* abort = &S.abort;

  if (warp == kExpWarps) {
    // ---------------------------------------------------------------- MMA issue
    if (lane == 0) {
      // D = f32, A = B = bf16, A K-major, B MN-major, N = n_pad, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (uint32_t(T.n_pad >> 3) << 17) |
                             (uint32_t(kRows >> 4) << 24);
      bool ok = true;
      for (int c = 0; c < n_chunks && !*abort; ++c) {
        const int s = c % kStages;
        const uint32_t ph = uint32_t(c / kStages) & 1u;
        if (!mbar_wait(smem_u32(&S.ops_full[s]), ph, abort, 22, T.status)) { ok = false; break; }
        tc_fence_after();
        const uint64_t de = smem_desc_sw128(smem_u32(S.e[s])), dq = smem_desc_sw128(smem_u32(S.o[s]));
        const uint64_t dv = smem_desc_sw128(smem_u32(S.v[s]), kVBlockBytes);
        const int keys_here = min(kKeys, k_end - c * kKeys);
        const int steps = (keys_here + 15) >> 4;                       // 16 keys per MMA
        for (int k = 0; k < steps; ++k) {
          const uint32_t accumulate = (c | k) != 0 ? 1u : 0u;
          umma_f16(tmem_base, de + uint64_t(2 * k), dv + uint64_t(128 * k), idesc, accumulate);
          umma_f16(tmem_base + uint32_t(T.n_pad), dq + uint64_t(2 * k), dv + uint64_t(128 * k), idesc, accumulate);
        }
        umma_commit(smem_u32(&S.ops_empty[s]));                        // stage free once these MMAs have read it
      }
      if (ok) umma_commit(smem_u32(&S.acc_full));
      // all MMAs issued by this thread must have completed before tensor memory is freed
      umma_commit(smem_u32(&S.done));
      mbar_drain(smem_u32(&S.done), 0);
    }
  } else {
    // ---------------------------------------------------------------- operand expansion
    const uint8_t* v_base = P.v + bo * P.v_so + bi * P.v_si;
    const float vz = __uint_as_float(kMagic) + float(P.z_v);           // exact: |z_v| is far below 2^22
    uint2 vraw[kVItems];
    auto fetch_v = [&](int c) {
#pragma unroll
      for (int q = 0; q < kVItems; ++q) {
        const int i = tid + kExpThreads * q;
        const int kr = i / (8 * NB), g = i % (8 * NB);
        const int key = c * kKeys + kr;
        vraw[q] = make_uint2(0u, 0u);
        if (c < n_chunks && key < P.Lk && g * 8 < P.d_h) {
          const uint8_t* src = v_base + int64_t(key) * P.ldv;
          if (P.bits_v == 4) vraw[q].x = __ldg(reinterpret_cast<const uint32_t*>(src + g * 4));
          else vraw[q] = __ldg(reinterpret_cast<const uint2*>(src + g * 8));
        }
      }
    };
    // this thread's codes of a chunk: 4 groups of 8 keys, group q = (row tid/8 + 32 q, keys 8 (tid%8) .. +7);
    // the 8 lanes of a row read its 32 or 64 contiguous code bytes
    const uint8_t* p_base = P.p + int64_t(pair) * P.p_pair;
    uint2 craw[4];
    auto fetch_codes = [&](int c) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = tid + kExpThreads * q;
        const int row = q0 + (i >> 3);
        const int64_t boff = int64_t(c) * kCodeBox + (i & 7) * (kCodeBox / 8);
        craw[q] = make_uint2(0u, 0u);
        if (c < n_chunks && row < P.Lq && boff + kCodeBox / 8 <= P.ldp) {
          const uint8_t* src = p_base + int64_t(row) * P.ldp + boff;
          if (kP4) craw[q].x = __ldcs(reinterpret_cast<const uint32_t*>(src));
          else craw[q] = __ldcs(reinterpret_cast<const uint2*>(src));
        }
      }
    };
    fetch_codes(0);
    fetch_v(0);
    for (int c = 0; c < n_chunks && !*abort; ++c) {
      const int s = c % kStages;
      const uint32_t ph = uint32_t(c / kStages) & 1u;
      const int k0 = c * kKeys;
      uint2 cw[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) cw[q] = craw[q];
      fetch_codes(c + 1);                                              // next chunk's codes, in flight meanwhile
      if (!mbar_wait(smem_u32(&S.ops_empty[s]), ph ^ 1u, abort, 24, T.status)) break;
      // ---- E and O tiles
      const bool masked = k0 + kKeys > min_valid;                      // CTA-uniform: some row ends inside this chunk
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = tid + kExpThreads * q;
        const int r = i >> 3, j = i & 7;
        uint4 ev, ov;
        if (kP4) {
          const uint2* lut = reinterpret_cast<const uint2*>(S.lut);
          const uint32_t w = cw[q].x;
          const uint2 a = lut[w & 0xFFu], b = lut[(w >> 8) & 0xFFu], c2 = lut[(w >> 16) & 0xFFu], d = lut[w >> 24];
          ev = make_uint4(a.x, b.x, c2.x, d.x);
          ov = make_uint4(a.y, b.y, c2.y, d.y);
        } else {
          const uint32_t* lut = S.lut;
          const uint32_t w0 = cw[q].x, w1 = cw[q].y;
          const uint32_t l0 = lut[w0 & 0xFFu], l1 = lut[(w0 >> 8) & 0xFFu], l2 = lut[(w0 >> 16) & 0xFFu], l3 = lut[w0 >> 24];
          const uint32_t l4 = lut[w1 & 0xFFu], l5 = lut[(w1 >> 8) & 0xFFu], l6 = lut[(w1 >> 16) & 0xFFu], l7 = lut[w1 >> 24];
          ev = make_uint4(__byte_perm(l0, l1, 0x5410), __byte_perm(l2, l3, 0x5410), __byte_perm(l4, l5, 0x5410), __byte_perm(l6, l7, 0x5410));
          ov = make_uint4(__byte_perm(l0, l1, 0x7632), __byte_perm(l2, l3, 0x7632), __byte_perm(l4, l5, 0x7632), __byte_perm(l6, l7, 0x7632));
        }
        if (masked) {
          const int row = q0 + r;
          const int valid = P.causal ? max(0, min(P.Lk, row + 1 + shift)) : P.Lk;
          const int limit = valid - (k0 + 8 * j);
          if (limit < 8) { keep_first(ev, limit); keep_first(ov, limit); }
        }
        const uint32_t off = tile_offset(r, j);
        *reinterpret_cast<uint4*>(S.e[s] + off) = ev;
        *reinterpret_cast<uint4*>(S.o[s] + off) = ov;
      }
      // ---- V tile: [key][channel] rows of 64 bf16 (v - z_v), zero rows past Lk, zero channels past d_h
#pragma unroll
      for (int q = 0; q < kVItems; ++q) {
        const int i = tid + kExpThreads * q;
        const int kr = i / (8 * NB), g = i % (8 * NB);
        uint32_t o4[4] = {0u, 0u, 0u, 0u};
        if (k0 + kr < P.Lk && g * 8 < P.d_h) {
          float f[8];
          if (P.bits_v == 4) {
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(kMagic | ((vraw[q].x >> (4 * e)) & 15u)) - vz;
          } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              f[e] = __uint_as_float(__byte_perm(vraw[q].x, kMagic, 0x7650 + e)) - vz;
              f[4 + e] = __uint_as_float(__byte_perm(vraw[q].y, kMagic, 0x7650 + e)) - vz;
            }
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
            o4[e] = *reinterpret_cast<const uint32_t*>(&h);
          }
        }
        *reinterpret_cast<uint4*>(S.v[s] + uint32_t(g >> 3) * kVBlockBytes + tile_offset(kr, g & 7)) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
      }
      fetch_v(c + 1);                                                  // next chunk's V rows, in flight meanwhile
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.ops_full[s]));
    }

    // ---------------------------------------------------------------- epilogue (warps 0..3: one row per thread)
    if (warp < 4 && !*abort && mbar_wait(smem_u32(&S.acc_full), 0, abort, 25, T.status)) {
      tc_fence_after();
      const float kSqrt2 = 1.41421356237309504880f;
      const float zo_lo = float(-P.zo), zo_hi = float(P.qmax - P.zo);
      const int r = warp * 32 + lane, row = q0 + r;
      const bool row_ok = row < P.Lq;
      const int64_t roff = bo * P.o_so + bi * P.o_si + int64_t(row) * P.ldo;
      const uint32_t taddr = tmem_base + (uint32_t(warp * 32) << 16);
      int code_sum = 0;
      for (int c0 = 0; c0 < P.d_h; c0 += 16) {
        uint32_t re[16], ro[16];
        __syncwarp();
        tmem_ld16(taddr + uint32_t(c0), re);
        tmem_ld16(taddr + uint32_t(T.n_pad + c0), ro);
        tmem_ld_wait();
        float v[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = P.scale * fmaf(kSqrt2, __uint_as_float(ro[e]), __uint_as_float(re[e]));
        if (!row_ok) continue;
        if (P.out_kind == REPQ_OUT_F32) {
          float* o = static_cast<float*>(P.out) + roff + c0;
          if (T.vec_store) {
#pragma unroll
            for (int e = 0; e < 4; ++e) reinterpret_cast<float4*>(o)[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = v[e];
          }
        } else if (P.out_kind == REPQ_OUT_BF16) {
          __nv_bfloat16* o = static_cast<__nv_bfloat16*>(P.out) + roff + c0;
          uint32_t w[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
            w[e] = *reinterpret_cast<const uint32_t*>(&h);
          }
          if (T.vec_store) {
            reinterpret_cast<uint4*>(o)[0] = make_uint4(w[0], w[1], w[2], w[3]);
            reinterpret_cast<uint4*>(o)[1] = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float2bfloat16_rn(v[e]);
          }
        } else {
          uint32_t q[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float tq = fminf(fmaxf(v[e] * P.inv_so, zo_lo), zo_hi);
            q[e] = uint32_t(__float2int_rn(tq) + P.zo);
            code_sum += int(q[e]);
          }
          uint8_t* orow = static_cast<uint8_t*>(P.out) + roff;
          if (P.pack4) {
            uint32_t w0 = 0u, w1 = 0u;
#pragma unroll
            for (int e = 0; e < 8; ++e) { w0 |= q[e] << (4 * e); w1 |= q[8 + e] << (4 * e); }
            if (T.vec_store) *reinterpret_cast<uint2*>(orow + (c0 >> 1)) = make_uint2(w0, w1);
            else {
#pragma unroll
              for (int e = 0; e < 4; ++e) { orow[(c0 >> 1) + e] = uint8_t(w0 >> (8 * e)); orow[(c0 >> 1) + 4 + e] = uint8_t(w1 >> (8 * e)); }
            }
          } else {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w[e] = q[4 * e] | (q[4 * e + 1] << 8) | (q[4 * e + 2] << 16) | (q[4 * e + 3] << 24);
            if (T.vec_store) *reinterpret_cast<uint4*>(orow + c0) = make_uint4(w[0], w[1], w[2], w[3]);
            else {
#pragma unroll
              for (int e = 0; e < 16; ++e) orow[c0 + e] = uint8_t(q[e]);
            }
          }
        }
      }
      if (P.out_row_sum != nullptr && P.out_kind == REPQ_OUT_CODES && row_ok)
        atomicAdd(P.out_row_sum + int64_t(bo) * P.Lq + row, code_sum);
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == kExpWarps) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(T.tmem_cols)) : "memory");
  }
}

template <bool kP4, int NB>
repq_status launch(const PvTcParams& T, const repq_pv_desc& d, int64_t pairs, cudaStream_t st) {
  using Shared = PvShared<kP4, NB>;
  const size_t smem = sizeof(Shared);
  REPQ_CUDA(cudaFuncSetAttribute(pv_tc_kernel<kP4, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  dim3 grid((d.Lq + kRows - 1) / kRows, unsigned(pairs));
  pv_tc_kernel<kP4, NB><<<grid, kThreads, smem, st>>>(T);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace

bool pv_tc_supported(const repq_pv_desc& d) {
  static const bool disabled = [] { const char* e = std::getenv("REPQ_DISABLE_TC"); return e && e[0] == '1'; }();
  if (disabled) return false;
  const int64_t unit = packed4(d.bits_v) ? 4 : 8;                    // bytes of 8 V codes: one vector load
  if (!aligned(d.v_codes, size_t(unit)) || d.ldv_bytes % unit || d.v_stride_outer % unit || d.v_stride_inner % unit) return false;
  return true;
}

repq_status launch_pv_tc(const repq_pv_desc& d, const PvParams& P, cudaStream_t st) {
  PvTcParams T{};
  T.p = P;
  T.n_pad = (d.d_h + 15) / 16 * 16;
  int cols = 32;
  while (cols < 2 * T.n_pad) cols *= 2;
  T.tmem_cols = cols;
  const int64_t esz = d.out_kind == REPQ_OUT_F32 ? 4 : d.out_kind == REPQ_OUT_BF16 ? 2 : 1;
  const int64_t chunk_bytes = d.out_kind == REPQ_OUT_CODES && packed4(d.out_bits) ? 8 : 16 * esz;   // bytes of 16 outputs
  const int64_t al = chunk_bytes < 16 ? chunk_bytes : 16;
  T.vec_store = aligned(d.out, size_t(al)) && (d.ldo * esz) % al == 0 && (d.o_stride_outer * esz) % al == 0 &&
                (d.o_stride_inner * esz) % al == 0;
  T.status = device_status_word();
  REPQ_REQUIRE(T.status != nullptr, REPQ_CUDA_ERROR, "pv: device status word unavailable");
  const int64_t pairs = int64_t(d.batch_outer) * d.batch_inner;
  const bool p4 = packed4(d.bits_p);
  if (d.d_h <= 64) return p4 ? launch<true, 1>(T, d, pairs, st) : launch<false, 1>(T, d, pairs, st);
  return p4 ? launch<true, 2>(T, d, pairs, st) : launch<false, 2>(T, d, pairs, st);
}

}  // namespace repq
