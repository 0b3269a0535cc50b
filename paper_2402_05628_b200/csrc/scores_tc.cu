// Attention scores S = alpha s_q s_k (Q - z_q)(K - z_k)^T per (batch, head) on integer codes (Eq. 3 with
// quantized Q and K) on the 5th-generation tensor cores, written as float32 rows for the Softmax stage.
//
// The contraction is only as long as the head (<= 128), so the kernel lives on its float32 writes.  A CTA owns
// 128 query rows of one (batch, head) pair and walks the keys in blocks of 128:
//   warps 0..7          copy the block's K codes (one code per byte; two threads per key, fetched one block ahead
//                       into registers) into a K-major, 128-byte-swizzled tile, with the keys' code sums for the
//                       zero-point correction; then the epilogue of the previous block: tcgen05.ld of the int32
//                       accumulator (one row per thread; warps 0..3 take columns 0..63, warps 4..7 columns 64..127),
//                       corr = acc - z_k qsum - z_q ksum + d_h z_q z_k, float32 scale, and out through a per-warp
//                       staging box of 32 rows x 128 bytes and a bulk tensor store (the 4-D tensor map clips rows
//                       past Lq and keys past Lk)
//   warp 8 (one lane)   tensor-memory allocation and MMA issue (kind::i8, u8 x u8 -> s32, N = 128); accumulators
//                       double-buffered in tensor memory so that the epilogue of block i overlaps block i + 1
// Under a causal mask, key blocks that no row of the CTA may see are skipped.
// Every mbarrier wait is bounded; when one runs out the kernel records a status code, all roles leave their
// loops, MMAs and stores in flight are drained, tensor memory is freed and the kernel returns.
#include <cstdlib>

#include "kernels.h"
#include "tc_ptx.cuh"

namespace repq {
namespace {

using namespace tc;

constexpr int kTile = 128;                 // query rows per CTA, keys per block
constexpr int kWorkWarps = 8;
constexpr int kWorkThreads = 32 * kWorkWarps;
constexpr int kThreads = kWorkThreads + 32;
constexpr uint32_t kTileBytes = kTile * 128;   // rows of 128 bytes (the head's codes, zero-padded)
constexpr int kTmemCols = 256;                 // two accumulators of 128 columns

struct ScoresTcParams {
  const uint8_t* q; const uint8_t* k;
  int64_t ldq, ldk, q_so, q_si, k_so, k_si;
  int Lq, Lk, dh, batch_inner;
  float scale;
  int zq, zk;
  int causal;
  int32_t* status;
};

struct ScoresShared {
  alignas(1024) uint8_t q[kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t box[kWorkWarps][4096];     // per-warp staging box: 32 rows x 32 floats
  int row_term[kTile];                             // -z_k qsum[m] + d_h z_q z_k
  int col_term[4][kTile];                          // -z_q ksum[n], ring of 4 key blocks
  alignas(8) uint64_t k_full[2];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t done;
  uint32_t tmem_base;
  volatile int abort;
};

__device__ __forceinline__ uint32_t tile_offset(int row, int piece) {
  return uint32_t(row >> 3) * 1024u + uint32_t(row & 7) * 128u + (uint32_t(piece ^ (row & 7)) << 4);
}

__device__ __forceinline__ int sum_bytes(const uint4& v) {
  return __dp4a(v.x, 0x01010101u, __dp4a(v.y, 0x01010101u, __dp4a(v.z, 0x01010101u, __dp4a(v.w, 0x01010101u, 0u))));
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int x, int y, int z, int w) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

__global__ void __launch_bounds__(kThreads)
scores_tc_kernel(const __grid_constant__ CUtensorMap map_out, ScoresTcParams P) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  ScoresShared& S = *reinterpret_cast<ScoresShared*>(smem_raw);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int pair = blockIdx.y;
  const int bo = pair / P.batch_inner, bi = pair % P.batch_inner;
  const int q0 = blockIdx.x * kTile;
  const int shift = P.Lk - P.Lq;
  const int k_end = P.causal ? max(1, min(P.Lk, min(q0 + kTile, P.Lq) + shift)) : P.Lk;
  const int n_blocks = (k_end + kTile - 1) / kTile;
  const int ksteps = (P.dh + 31) >> 5;                   // MMAs of K = 32 per key block
  const int pieces = P.dh >> 4;                          // 16-byte pieces of a row (d_h is a multiple of 16)

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&S.k_full[s]), kWorkWarps);
      mbar_init(smem_u32(&S.acc_full[s]), 1);
      mbar_init(smem_u32(&S.acc_empty[s]), kWorkWarps);
    }
    mbar_init(smem_u32(&S.done), 1);
    S.abort = 0;
    if (smem_u32(smem_raw) & 1023u) {                    // the swizzled tiles need this alignment
      atomicCAS(P.status, 0, 39);
      S.abort = 1;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWorkWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&S.tmem_base)), "n"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  // Two threads per row: thread (row, half) owns pieces 4 half .. 4 half + 3 of the row's (up to 8) pieces.
  const int lrow = (tid >> 1) & (kTile - 1), lhalf = tid & 1;
  uint4 kreg[4];
  auto fetch_rows = [&](const uint8_t* base, int64_t ld, int r0, int rows, uint4 (&dst)[4]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      dst[j] = make_uint4(0u, 0u, 0u, 0u);
      const int piece = 4 * lhalf + j;
      if (r0 + lrow < rows && piece < pieces)
        dst[j] = __ldg(reinterpret_cast<const uint4*>(base + int64_t(r0 + lrow) * ld) + piece);
    }
  };
  // writes the thread's pieces into a tile and returns the code sum of its whole row
  auto store_rows = [&](uint8_t* tile, const uint4 (&src)[4]) {
    int s = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int piece = 4 * lhalf + j;
      if (piece < 2 * ksteps) *reinterpret_cast<uint4*>(tile + tile_offset(lrow, piece)) = src[j];
      s += sum_bytes(src[j]);
    }
    return s + __shfl_xor_sync(0xffffffffu, s, 1);
  };

  if (warp < kWorkWarps) {
    // Q tile and its row terms, once per CTA
    uint4 qreg[4];
    fetch_rows(P.q + bo * P.q_so + bi * P.q_si, P.ldq, q0, P.Lq, qreg);
    fetch_rows(P.k + bo * P.k_so + bi * P.k_si, P.ldk, 0, P.Lk, kreg);
    const int qs = store_rows(S.q, qreg);
    if (lhalf == 0) S.row_term[lrow] = -P.zk * qs + P.dh * P.zq * P.zk;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S.tmem_base;
  volatile int* abort = &S.abort;

  if (warp == kWorkWarps) {
    // ---------------------------------------------------------------- MMA issue
    if (lane == 0) {
      // D = s32, A = B = unsigned 8-bit, both K-major, N = 128, M = 128
      constexpr uint32_t idesc = (2u << 4) | (uint32_t(kTile >> 3) << 17) | (uint32_t(kTile >> 4) << 24);
      const uint64_t dq = smem_desc_sw128(smem_u32(S.q));
      for (int kb = 0; kb < n_blocks && !*abort; ++kb) {
        const int b = kb & 1;
        const uint32_t ph = uint32_t(kb >> 1) & 1u;
        if (!mbar_wait(smem_u32(&S.k_full[b]), ph, abort, 31, P.status)) break;
        if (!mbar_wait(smem_u32(&S.acc_empty[b]), ph ^ 1u, abort, 32, P.status)) break;
        tc_fence_after();
        const uint64_t dk = smem_desc_sw128(smem_u32(S.k[b]));
        for (int s = 0; s < ksteps; ++s)
          umma_i8(tmem_base + uint32_t(b * kTile), dq + uint64_t(2 * s), dk + uint64_t(2 * s), idesc, s != 0 ? 1u : 0u);
        umma_commit(smem_u32(&S.acc_full[b]));
      }
      // all MMAs issued by this thread must have completed before tensor memory is freed
      umma_commit(smem_u32(&S.done));
      mbar_drain(smem_u32(&S.done), 0);
    }
  } else {
    // ---------------------------------------------------------------- K tiles and epilogue
    const int quarter = warp & 3, half = warp >> 2;
    const int row = q0 + quarter * 32 + lane;
    const uint32_t box = smem_u32(S.box[warp]);
    const int my_row_term = S.row_term[quarter * 32 + lane];
    const bool rows_live = q0 + quarter * 32 < P.Lq;            // warp-uniform: the box has a row inside the matrix
    const int last_key = P.causal ? min(P.Lk, q0 + quarter * 32 + 32 + shift) : P.Lk;   // keys the warp's rows may see

    auto epilogue = [&](int kb) -> bool {
      const int b = kb & 1;
      if (!mbar_wait(smem_u32(&S.acc_full[b]), uint32_t(kb >> 1) & 1u, abort, 33, P.status)) return false;
      tc_fence_after();
      const int* ct = S.col_term[kb & 3];
#pragma unroll 1
      for (int g = 0; g < 2; ++g) {
        const int c0 = half * 64 + g * 32;                      // first column of the box inside the key block
        const int n0 = kb * kTile + c0;
        if (!rows_live || n0 >= last_key) continue;             // warp-uniform
        uint32_t r0[16], r1[16];
        __syncwarp();
        tmem_ld16(tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(b * kTile + c0), r0);
        tmem_ld16(tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(b * kTile + c0 + 16), r1);
        tmem_ld_wait();
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the box is free again
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int4 c4 = *reinterpret_cast<const int4*>(ct + c0 + 4 * j);
          const uint32_t* r = j < 4 ? &r0[4 * j] : &r1[4 * (j - 4)];
          float4 v;
          v.x = P.scale * float(int32_t(r[0]) + my_row_term + c4.x);
          v.y = P.scale * float(int32_t(r[1]) + my_row_term + c4.y);
          v.z = P.scale * float(int32_t(r[2]) + my_row_term + c4.z);
          v.w = P.scale * float(int32_t(r[3]) + my_row_term + c4.w);
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                       ::"r"(box + uint32_t(lane) * 128u + (uint32_t(j ^ (lane & 7)) << 4)), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_4d(&map_out, box, n0, q0 + quarter * 32, bi, bo);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      (void)row;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.acc_empty[b]));
      return true;
    };

    const uint8_t* k_base = P.k + bo * P.k_so + bi * P.k_si;
    bool ok = true;
    for (int kb = 0; kb < n_blocks && !*abort; ++kb) {
      // tile kb & 1 was last read by the MMAs of block kb - 2, whose accumulator this thread has already waited for
      const int ks = store_rows(S.k[kb & 1], kreg);
      if (lhalf == 0) S.col_term[kb & 3][lrow] = -P.zq * ks;
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.k_full[kb & 1]));
      if (kb + 1 < n_blocks) fetch_rows(k_base, P.ldk, (kb + 1) * kTile, P.Lk, kreg);   // in flight during the epilogue
      if (kb > 0 && !epilogue(kb - 1)) { ok = false; break; }
    }
    if (ok && !*abort) epilogue(n_blocks - 1);
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");            // bulk stores complete
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == kWorkWarps) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
  }
}

}  // namespace

bool scores_tc_supported(const repq_gemm_desc& d) {
  static const bool disabled = [] { const char* e = std::getenv("REPQ_DISABLE_TC"); return e && e[0] == '1'; }();
  if (disabled) return false;
  if (packed4(d.bits_a) || packed4(d.bits_w)) return false;             // one code per byte on both sides
  if (d.K % 16 != 0 || d.K > 128) return false;
  auto ok = [&](const void* p, int64_t ld, int64_t so, int64_t si) {
    return aligned(p, 16) && ld % 16 == 0 && so % 16 == 0 && si % 16 == 0;
  };
  if (!ok(d.a_codes, d.lda_bytes, d.a_stride_outer, d.a_stride_inner)) return false;
  if (!ok(d.w_codes, d.ldw_bytes, d.w_stride_outer, d.w_stride_inner)) return false;
  // output rows as a 4-D tensor (key, query, inner batch, outer batch): 16-byte strides, extents the map can hold
  if (!aligned(d.out, 16) || d.ldo % 4 != 0 || d.o_stride_outer % 4 != 0 || d.o_stride_inner % 4 != 0) return false;
  if (d.batch_inner > 1 && d.o_stride_inner <= 0) return false;
  if (d.batch_outer > 1 && d.o_stride_outer <= 0) return false;
  if (int64_t(d.batch_outer) * d.batch_inner > 65535) return false;
  return true;
}

repq_status launch_scores_tc(const repq_gemm_desc& d, cudaStream_t st) {
  EncodeTiledFn fn = encode_fn();
  REPQ_REQUIRE(fn != nullptr, REPQ_CUDA_ERROR, "qgemm: cuTensorMapEncodeTiled is not available");
  const int64_t row_bytes = int64_t(d.ldo) * 4;
  const cuuint64_t dims[4] = {cuuint64_t(d.N), cuuint64_t(d.M), cuuint64_t(d.batch_inner), cuuint64_t(d.batch_outer)};
  const cuuint64_t strides[3] = {cuuint64_t(row_bytes),
                                 cuuint64_t(d.batch_inner > 1 ? d.o_stride_inner * 4 : row_bytes * d.M),
                                 cuuint64_t(d.batch_outer > 1 ? d.o_stride_outer * 4 : row_bytes * d.M * d.batch_inner)};
  const cuuint32_t box[4] = {32, 32, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  CUtensorMap map;
  const CUresult r = fn(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, d.out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  REPQ_REQUIRE(r == CUDA_SUCCESS, REPQ_CUDA_ERROR, "qgemm: scores tensor map failed with code %d", int(r));
  ScoresTcParams P{};
  P.q = d.a_codes; P.k = d.w_codes;
  P.ldq = d.lda_bytes; P.ldk = d.ldw_bytes;
  P.q_so = d.a_stride_outer; P.q_si = d.a_stride_inner; P.k_so = d.w_stride_outer; P.k_si = d.w_stride_inner;
  P.Lq = d.M; P.Lk = d.N; P.dh = d.K; P.batch_inner = d.batch_inner;
  P.scale = d.alpha * d.s_a * d.s_w_scalar;
  P.zq = d.z_a; P.zk = d.z_w_scalar;
  P.causal = d.causal;
  P.status = device_status_word();
  REPQ_REQUIRE(P.status != nullptr, REPQ_CUDA_ERROR, "qgemm: device status word unavailable");
  const size_t smem = sizeof(ScoresShared);
  REPQ_CUDA(cudaFuncSetAttribute(scores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  dim3 grid((d.M + kTile - 1) / kTile, unsigned(int64_t(d.batch_outer) * d.batch_inner));
  scores_tc_kernel<<<grid, kThreads, smem, st>>>(map, P);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace repq
