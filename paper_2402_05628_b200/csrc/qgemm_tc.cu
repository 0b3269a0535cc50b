// Integer GEMM on the 5th-generation tensor cores: TMA-fed shared-memory operand ring, single-thread
// tcgen05.mma (kind::i8, u8 x u8 -> s32) into tensor memory, and an epilogue that reads the int32
// accumulators back with tcgen05.ld and applies the zero-point correction, scale, bias, GELU, residual
// and re-quantization of the quantized linear layer.
//
// One persistent CTA per SM; roles by warp:
//   warp 0      TMA producer (one elected lane): A tile 128 x 128 B, W tile 256 x 128 B per stage, 128-byte
//               swizzle, zero fill outside the matrices
//   warp 1      tensor-memory allocation and MMA issue (one elected lane): 4 MMAs of K = 32 per stage,
//               accumulators double-buffered in TMEM (2 x 256 columns) so the epilogue of tile i overlaps
//               the main loop of tile i + 1
//   warps 2..9  epilogue: warp w reads TMEM lanes 32 (w mod 4) .. +31 (one output row per thread) and one
//               half of the 256 accumulator columns
// 4-bit operands are expanded to one code per byte by a separate pass into the workspace (there is no
// 4-bit integer MMA), so the main loop is the same for W4A4 and W8A8.
//
// Every wait on an mbarrier is bounded: when it runs out the kernel records a status code, all roles
// leave their loops, in-flight copies and MMAs are drained, tensor memory is freed and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>
#include <mutex>

#include "kernels.h"

namespace repq {
namespace {

constexpr int BM = 128, BN = 256, BK = 128;        // BK in bytes (= codes)
constexpr int kStages = 4;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;
constexpr uint32_t kABytes = BM * BK, kBBytes = BN * BK;
constexpr long long kWaitCycles = 2000000000LL;     // about one second

__device__ int32_t g_status_word = 0;

struct alignas(16) ColTerms {                         // per output column, staged once per tile
  float scale[BN];
  float bias[BN];
  int32_t z_w[BN];
  int32_t kzz[BN];
  float inv_so[BN];
  int32_t zo[BN];
};

struct SharedStorage {
  alignas(1024) uint8_t a[kStages][kABytes];
  alignas(1024) uint8_t b[kStages][kBBytes];
  ColTerms cols[2];
  alignas(8) uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t cols_ready[2];
  uint64_t done;
  uint32_t tmem_base;
  volatile int abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Bounded wait: false if the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort) return false;
    if (clock64() - t0 > kWaitCycles) {
      atomicCAS(&g_status_word, 0, code);
      *abort = 1;
      return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 256 x 32, u8 x u8 -> s32
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory matrix descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return uint64_t((addr >> 4) & 0x3FFFu) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) |
         (uint64_t(2) << 61);
}

// Instruction descriptor: D = s32, A = B = unsigned 8-bit, both K-major, N = 256, M = 128.
constexpr uint32_t kIdesc = (2u << 4) | (0u << 7) | (0u << 10) | (uint32_t(BN >> 3) << 17) | (uint32_t(BM >> 4) << 24);

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

struct TcParams {
  int M, N, K;
  const int32_t* asum;
  const int32_t* wsum;
  EpilogueParams ep;
};

__global__ void __launch_bounds__(kThreads, 1)
qgemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, TcParams P) {
  extern __shared__ uint8_t smem_raw[];
  SharedStorage& S = *reinterpret_cast<SharedStorage*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (P.M + BM - 1) / BM, n_tiles = (P.N + BN - 1) / BN;
  const int tiles = m_tiles * n_tiles;
  const int kblocks = (P.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&S.full[s]), 1); mbar_init(smem_u32(&S.empty[s]), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&S.tmem_full[a]), 1); mbar_init(smem_u32(&S.tmem_empty[a]), kEpiWarps); }
    for (int a = 0; a < 2; ++a) mbar_init(smem_u32(&S.cols_ready[a]), kEpiWarps * 32);
    mbar_init(smem_u32(&S.done), 1);
    S.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&S.tmem_base)), "n"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S.tmem_base;
  volatile int* abort = &S.abort;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      long long issued = 0;
      for (int tile = blockIdx.x; tile < tiles && !*abort; tile += gridDim.x) {
        const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(smem_u32(&S.empty[stage]), phase ^ 1, abort, 1)) break;
          const uint32_t bar = smem_u32(&S.full[stage]);
          mbar_expect_tx(bar, kABytes + kBBytes);
          tma_load_2d(smem_u32(S.a[stage]), &map_a, bar, kb * BK, m0);
          tma_load_2d(smem_u32(S.b[stage]), &map_b, bar, kb * BK, n0);
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      // drain: the copies issued last must have landed before this CTA may exit
      const int back = issued < kStages ? int(issued) : kStages;
      uint32_t s = stage, ph = phase;
      for (int i = 0; i < back; ++i) {
        if (s == 0) { s = kStages - 1; ph ^= 1; } else { --s; }
        const long long t0 = clock64();
        while (!mbar_try_wait(smem_u32(&S.full[s]), ph) && clock64() - t0 < kWaitCycles) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issue
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      int it = 0;
      for (int tile = blockIdx.x; tile < tiles && !*abort; tile += gridDim.x, ++it) {
        const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
        if (!mbar_wait(smem_u32(&S.tmem_empty[acc]), acc_phase ^ 1, abort, 2)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        bool ok = true;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(smem_u32(&S.full[stage]), phase, abort, 3)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = smem_desc(smem_u32(S.a[stage])), db = smem_desc(smem_u32(S.b[stage]));
#pragma unroll
          for (int k = 0; k < BK / 32; ++k)
            umma_i8(d_tmem, da + uint64_t(k * 2), db + uint64_t(k * 2), kIdesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(smem_u32(&S.empty[stage]));          // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&S.tmem_full[acc]));           // accumulator complete
      }
      // all MMAs issued by this thread must have completed before tensor memory is freed
      umma_commit(smem_u32(&S.done));
      const long long t0 = clock64();
      while (!mbar_try_wait(smem_u32(&S.done), 0) && clock64() - t0 < kWaitCycles) {}
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - 2;                     // 0..7
    const int quarter = warp & 3;                // TMEM lane quarter this warp may read
    const int half = ew >> 2;                    // which 128 accumulator columns
    const int et = threadIdx.x - 64;             // 0..255 among epilogue threads
    const EpilogueParams& ep = P.ep;
    int it = 0;
    for (int tile = blockIdx.x; tile < tiles && !*abort; tile += gridDim.x, ++it) {
      const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
      const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
      // stage the per-column terms of this tile (one column per epilogue thread); the buffer was last
      // read two tiles ago, before this thread's arrival on tmem_empty of that tile
      {
        ColTerms& C = S.cols[acc];
        const int j = n0 + et;
        if (j < P.N) {
          const ColumnTerms ct = column_terms(ep, j, __ldg(P.wsum + j));
          C.scale[et] = ct.scale; C.bias[et] = ct.bias; C.z_w[et] = ct.z_w; C.kzz[et] = ct.kzz;
          C.inv_so[et] = ct.inv_so; C.zo[et] = ct.zo;
        } else {
          C.scale[et] = 0.f; C.bias[et] = 0.f; C.z_w[et] = 0; C.kzz[et] = 0; C.inv_so[et] = 1.f; C.zo[et] = 0;
        }
        mbar_arrive(smem_u32(&S.cols_ready[acc]));           // release: orders the writes above
        if (!mbar_wait(smem_u32(&S.cols_ready[acc]), acc_phase, abort, 5)) break;
      }
      if (!mbar_wait(smem_u32(&S.tmem_full[acc]), acc_phase, abort, 4)) break;
      tc_fence_after();

      const int64_t m = int64_t(m0) + quarter * 32 + lane;
      const bool row_ok = m < P.M;
      const int32_t asum_m = row_ok ? __ldg(P.asum + m) : 0;
      const ColTerms& C = S.cols[acc];
      int code_sum = 0;
#pragma unroll 1
      for (int c = 0; c < (BN / 2) / 32; ++c) {
        const int cl = half * (BN / 2) + c * 32;          // column inside the tile
        uint32_t r[32];
        __syncwarp();
        tmem_ld32(tmem_base + (uint32_t(quarter * 32) << 16) + acc * BN + cl, r);
        tmem_ld_wait();
        const int col0 = n0 + cl;
        if (row_ok && col0 < P.N) {
        const bool full_chunk = col0 + 32 <= P.N;
        if (ep.acc_debug) {
          for (int e = 0; e < 32; ++e)
            if (col0 + e < P.N) ep.acc_debug[m * P.N + col0 + e] = int32_t(r[e]);
        }
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int32_t corr = int32_t(r[e] - uint32_t(C.z_w[cl + e]) * uint32_t(asum_m) + uint32_t(C.kzz[cl + e]));
          v[e] = fmaf(C.scale[cl + e], float(corr), C.bias[cl + e]);
        }
        if (ep.gelu) {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = gelu_erf(v[e]);
        }
        if (ep.residual) {
          if (ep.residual_bf16) {
            const __nv_bfloat16* rp = static_cast<const __nv_bfloat16*>(ep.residual) + m * ep.ld_residual + col0;
            if (full_chunk) {
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) {
                const uint4 w = __ldg(reinterpret_cast<const uint4*>(rp) + q4);
                const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  v[q4 * 8 + 2 * i] += __uint_as_float(ws[i] << 16);
                  v[q4 * 8 + 2 * i + 1] += __uint_as_float(ws[i] & 0xffff0000u);
                }
              }
            } else {
              for (int e = 0; e < 32; ++e) if (col0 + e < P.N) v[e] += __bfloat162float(rp[e]);
            }
          } else {
            const float* rp = static_cast<const float*>(ep.residual) + m * ep.ld_residual + col0;
            if (full_chunk) {
#pragma unroll
              for (int q4 = 0; q4 < 8; ++q4) {
                const float4 w = __ldg(reinterpret_cast<const float4*>(rp) + q4);
                v[q4 * 4] += w.x; v[q4 * 4 + 1] += w.y; v[q4 * 4 + 2] += w.z; v[q4 * 4 + 3] += w.w;
              }
            } else {
              for (int e = 0; e < 32; ++e) if (col0 + e < P.N) v[e] += rp[e];
            }
          }
        }
        if (ep.out_kind == REPQ_OUT_F32) {
          float* o = static_cast<float*>(ep.out) + m * ep.ldo + col0;
          if (full_chunk) {
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4)
              reinterpret_cast<float4*>(o)[q4] = make_float4(v[q4 * 4], v[q4 * 4 + 1], v[q4 * 4 + 2], v[q4 * 4 + 3]);
          } else {
            for (int e = 0; e < 32; ++e) if (col0 + e < P.N) o[e] = v[e];
          }
        } else if (ep.out_kind == REPQ_OUT_BF16) {
          __nv_bfloat16* o = static_cast<__nv_bfloat16*>(ep.out) + m * ep.ldo + col0;
          if (full_chunk) {
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              uint32_t w[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(v[q4 * 8 + 2 * i], v[q4 * 8 + 2 * i + 1]);
                w[i] = *reinterpret_cast<const uint32_t*>(&h);
              }
              reinterpret_cast<uint4*>(o)[q4] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          } else {
            for (int e = 0; e < 32; ++e) if (col0 + e < P.N) o[e] = __float2bfloat16_rn(v[e]);
          }
        } else {
          uint32_t q[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int zo = C.zo[cl + e];
            float t = v[e] * C.inv_so[cl + e];
            t = fminf(fmaxf(t, float(-zo)), float(ep.qmax - zo));
            q[e] = uint32_t(__float2int_rn(t) + zo);
            if (col0 + e >= P.N) q[e] = 0;
            code_sum += int(q[e]);
          }
          uint8_t* orow = static_cast<uint8_t*>(ep.out) + m * ep.ldo;
          if (ep.pack4) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              w[i] = 0;
#pragma unroll
              for (int e = 0; e < 8; ++e) w[i] |= q[i * 8 + e] << (4 * e);
            }
            if (full_chunk) {
              *reinterpret_cast<uint4*>(orow + (col0 >> 1)) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
              for (int e = 0; e < 32; e += 2)
                if (col0 + e < P.N) orow[(col0 + e) >> 1] = uint8_t(q[e] | (q[e + 1] << 4));
            }
          } else {
            if (full_chunk) {
#pragma unroll
              for (int h2 = 0; h2 < 2; ++h2) {
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int b = h2 * 16 + i * 4;
                  w[i] = q[b] | q[b + 1] << 8 | q[b + 2] << 16 | q[b + 3] << 24;
                }
                reinterpret_cast<uint4*>(orow + col0)[h2] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            } else {
              for (int e = 0; e < 32; ++e) if (col0 + e < P.N) orow[col0 + e] = uint8_t(q[e]);
            }
          }
        }
        }
      }
      // accumulator buffer free again
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.tmem_empty[acc]));
      if (ep.out_row_sum != nullptr && row_ok && code_sum != 0) atomicAdd(ep.out_row_sum + m, code_sum);
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
  }
}

// ---- host side -------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

repq_status make_map(CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t K, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  REPQ_REQUIRE(fn != nullptr, REPQ_CUDA_ERROR, "qgemm: cuTensorMapEncodeTiled is not available");
  const cuuint64_t dims[2] = {cuuint64_t(K), cuuint64_t(rows)};
  const cuuint64_t strides[1] = {cuuint64_t(ld)};
  const cuuint32_t box[2] = {cuuint32_t(BK), cuuint32_t(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  REPQ_REQUIRE(r == CUDA_SUCCESS, REPQ_CUDA_ERROR, "qgemm: cuTensorMapEncodeTiled failed with code %d", int(r));
  return REPQ_OK;
}

struct TcLayout {
  size_t off_a, off_w, off_asum, off_wsum, total;
  int64_t ld_a, ld_w;
};

TcLayout tc_layout(const repq_gemm_desc& d) {
  TcLayout L{};
  size_t cur = 0;
  auto bump = [&](size_t bytes) { size_t at = cur; cur += (bytes + 255) / 256 * 256; return at; };
  L.ld_a = round_up(d.K, 16);
  L.ld_w = round_up(d.K, 16);
  L.off_a = d.bits_a == 4 ? bump(size_t(d.M) * L.ld_a) : 0;
  L.off_w = d.bits_w == 4 ? bump(size_t(d.N) * L.ld_w) : 0;
  L.off_asum = d.a_row_sum ? 0 : bump(size_t(d.M) * 4);
  L.off_wsum = d.w_row_sum ? 0 : bump(size_t(d.N) * 4);
  L.total = cur;
  return L;
}

}  // namespace

int32_t* device_status_word() {
  static int32_t* addr[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    addr[dev] = static_cast<int32_t*>(p);
  }
  return addr[dev];
}

bool qgemm_tc_supported(const repq_gemm_desc& d) {
  static const bool disabled = [] { const char* e = std::getenv("REPQ_DISABLE_TC"); return e && e[0] == '1'; }();
  if (disabled) return false;
  if (d.batch_outer != 1 || d.batch_inner != 1) return false;
  if (d.M < 64 || d.N < 64 || d.K < 64) return false;           // tiny problems: the warp-MMA kernel
  if (d.bits_a != 4 && !(aligned(d.a_codes, 16) && d.lda_bytes % 16 == 0)) return false;
  if (d.bits_w != 4 && !(aligned(d.w_codes, 16) && d.ldw_bytes % 16 == 0)) return false;
  const int64_t obytes = d.out_kind == REPQ_OUT_F32 ? 4 : d.out_kind == REPQ_OUT_BF16 ? 2 : 1;
  if (!aligned(d.out, 16) || (d.ldo * obytes) % 16 != 0) return false;
  if (d.residual) {
    const int64_t rb = d.residual_dtype == REPQ_F32 ? 4 : 2;
    if (!aligned(d.residual, 16) || (d.ld_residual * rb) % 16 != 0) return false;
  }
  return true;
}

size_t qgemm_tc_workspace(const repq_gemm_desc& d) { return tc_layout(d).total; }

repq_status qgemm_tc(const repq_gemm_desc& d, const EpilogueParams& ep, void* ws, size_t ws_bytes, cudaStream_t st) {
  const TcLayout L = tc_layout(d);
  REPQ_REQUIRE(ws_bytes >= L.total, REPQ_WORKSPACE_TOO_SMALL, "qgemm: workspace too small");
  REPQ_REQUIRE(L.total == 0 || aligned(ws, 256), REPQ_ALIGNMENT, "qgemm: workspace must be 256-byte aligned");
  uint8_t* w8 = static_cast<uint8_t*>(ws);
  const uint8_t* a = d.a_codes;
  int64_t lda = d.lda_bytes;
  if (d.bits_a == 4) {
    REPQ_TRY(launch_expand4(d.a_codes, d.M, d.K, d.lda_bytes, w8 + L.off_a, L.ld_a, L.ld_a, st));
    a = w8 + L.off_a; lda = L.ld_a;
  }
  const uint8_t* w = d.w_codes;
  int64_t ldw = d.ldw_bytes;
  if (d.bits_w == 4) {
    REPQ_TRY(launch_expand4(d.w_codes, d.N, d.K, d.ldw_bytes, w8 + L.off_w, L.ld_w, L.ld_w, st));
    w = w8 + L.off_w; ldw = L.ld_w;
  }
  TcParams P{};
  P.M = d.M; P.N = d.N; P.K = d.K;
  P.asum = d.a_row_sum;
  if (!P.asum) {
    int32_t* s = reinterpret_cast<int32_t*>(w8 + L.off_asum);
    REPQ_TRY(launch_row_sum(d.a_codes, d.bits_a, d.M, d.K, d.lda_bytes, s, st));
    P.asum = s;
  }
  P.wsum = d.w_row_sum;
  if (!P.wsum) {
    int32_t* s = reinterpret_cast<int32_t*>(w8 + L.off_wsum);
    REPQ_TRY(launch_row_sum(d.w_codes, d.bits_w, d.N, d.K, d.ldw_bytes, s, st));
    P.wsum = s;
  }
  P.ep = ep;
  CUtensorMap map_a, map_b;
  REPQ_TRY(make_map(&map_a, a, d.M, d.K, lda, BM));
  REPQ_TRY(make_map(&map_b, w, d.N, d.K, ldw, BN));
  REPQ_REQUIRE(device_status_word() != nullptr, REPQ_CUDA_ERROR, "qgemm: device status word unavailable");

  const size_t smem = sizeof(SharedStorage) + 1024;
  REPQ_CUDA(cudaFuncSetAttribute(qgemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  const int m_tiles = (d.M + BM - 1) / BM, n_tiles = (d.N + BN - 1) / BN;
  const int tiles = m_tiles * n_tiles;
  const int sms = sm_count();
  const int grid = tiles < sms ? tiles : sms;
  qgemm_tc_kernel<<<grid, kThreads, smem, st>>>(map_a, map_b, P);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace repq
