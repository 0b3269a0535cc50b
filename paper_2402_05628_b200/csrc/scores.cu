// Attention scores S = s_q s_k alpha (Q - z_q)(K - z_k)^T per (batch, head) on integer codes (Eq. 3 with
// quantized Q and K), written as float32 rows for the Softmax stage.
//
// The contraction length is the head size (<= 128), so the kernel is bound by the float32 score writes:
// a CTA owns 128 query rows of one (batch, head) pair, keeps their codes in shared memory, walks the keys in
// tiles of 128, and multiplies with warp-level u8 MMA (m16n8k32).  Row sums of Q and K codes for the
// zero-point correction come from the same shared-memory tiles.  With `causal`, key tiles that lie
// entirely above the diagonal are skipped (their scores are never read).
#include "kernels.h"

namespace repq {
namespace {

constexpr int kTile = 128;                 // query rows per CTA, keys per step
constexpr int kThreads = 256;
constexpr int kMaxRowBytes = 128 + 16;     // padded shared-memory row (head size <= 128)

struct ScoresParams {
  const uint8_t* q; const uint8_t* k;
  int64_t ldq, ldk, q_so, q_si, k_so, k_si;
  int Lq, Lk, dh, dhp, batch_inner;
  float scale;
  int zq, zk;
  float* out; int64_t ldo, o_so, o_si;
  int causal;
};

__device__ __forceinline__ void mma_u8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Copies rows [r0, r0 + 128) of a code matrix (head slice of dh codes) into shared memory, one code per
// byte, zero beyond `rows` and beyond dh.  Work unit: 16 codes.
template <bool k4>
__device__ __forceinline__ void stage_tile(const uint8_t* base, int64_t ld, int r0, int rows, int dh, int dhp,
                                           uint8_t* smem, int row_bytes) {
  const int units_per_row = dhp / 16;
  for (int u = threadIdx.x; u < kTile * units_per_row; u += kThreads) {
    const int r = u / units_per_row, c = (u % units_per_row) * 16;
    uint4 o = make_uint4(0, 0, 0, 0);
    if (r0 + r < rows && c < dh) {
      const uint8_t* src = base + int64_t(r0 + r) * ld;
      if (k4) {
        const uint2 w = *reinterpret_cast<const uint2*>(src + c / 2);
        uint32_t lo = w.x & 0x0F0F0F0Fu, hi = (w.x >> 4) & 0x0F0F0F0Fu;
        o.x = __byte_perm(lo, hi, 0x5140); o.y = __byte_perm(lo, hi, 0x7362);
        lo = w.y & 0x0F0F0F0Fu; hi = (w.y >> 4) & 0x0F0F0F0Fu;
        o.z = __byte_perm(lo, hi, 0x5140); o.w = __byte_perm(lo, hi, 0x7362);
      } else {
        o = *reinterpret_cast<const uint4*>(src + c);
      }
    }
    *reinterpret_cast<uint4*>(smem + r * row_bytes + c) = o;
  }
}

// term[r] = -mult * (sum of the codes of row r)
__device__ __forceinline__ void row_terms(const uint8_t* smem, int row_bytes, int dhp, int mult, int* term, int idx) {
  if (idx >= 0 && idx < kTile) {
    const uint32_t* p = reinterpret_cast<const uint32_t*>(smem + idx * row_bytes);
    int s = 0;
    for (int i = 0; i < dhp / 4; ++i) s = __dp4a(p[i], 0x01010101u, uint32_t(s));
    term[idx] = -mult * s;
  }
}

template <bool k4>
__global__ void __launch_bounds__(kThreads, 3)
scores_kernel(ScoresParams P) {
  __shared__ __align__(16) uint8_t sQ[kTile * kMaxRowBytes];
  __shared__ __align__(16) uint8_t sK[kTile * kMaxRowBytes];
  __shared__ int q_term[kTile];
  __shared__ int k_term[kTile];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int pair = blockIdx.y, bo = pair / P.batch_inner, bi = pair % P.batch_inner;
  const int q0 = blockIdx.x * kTile;
  const int row_bytes = P.dhp + 16;
  const uint8_t* qb = P.q + bo * P.q_so + bi * P.q_si;
  const uint8_t* kb = P.k + bo * P.k_so + bi * P.k_si;
  float* ob = P.out + bo * P.o_so + bi * P.o_si;

  stage_tile<k4>(qb, P.ldq, q0, P.Lq, P.dh, P.dhp, sQ, row_bytes);
  __syncthreads();
  row_terms(sQ, row_bytes, P.dhp, P.zk, q_term, tid);          // -z_k * sum_d q[i, d]

  const int wr = (warp & 3) * 32, wc = (warp >> 2) * 64;        // warp tile: 32 rows x 64 keys
  const int g = lane >> 2, t = lane & 3;
  const int shift = P.Lk - P.Lq;
  int k_end = P.Lk;
  if (P.causal) k_end = max(0, min(P.Lk, min(q0 + kTile, P.Lq) + shift));
  const int kzz = P.dh * P.zq * P.zk;

  for (int k0 = 0; k0 < k_end; k0 += kTile) {
    __syncthreads();                                             // previous tile fully consumed
    stage_tile<k4>(kb, P.ldk, k0, P.Lk, P.dh, P.dhp, sK, row_bytes);
    __syncthreads();
    row_terms(sK, row_bytes, P.dhp, P.zq, k_term, tid - kTile);     // -z_q * sum_d k[j, d], by the upper 128 threads
    int acc[2][8][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][j][e] = 0;
    for (int ks = 0; ks < P.dhp; ks += 32) {
      uint32_t af[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint8_t* p = sQ + (wr + i * 16 + g) * row_bytes + ks + 4 * t;
        af[i][0] = *reinterpret_cast<const uint32_t*>(p);
        af[i][1] = *reinterpret_cast<const uint32_t*>(p + 8 * row_bytes);
        af[i][2] = *reinterpret_cast<const uint32_t*>(p + 16);
        af[i][3] = *reinterpret_cast<const uint32_t*>(p + 8 * row_bytes + 16);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint8_t* p = sK + (wc + j * 8 + g) * row_bytes + ks + 4 * t;
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(p);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(p + 16);
        mma_u8(acc[0][j], af[0], b0, b1);
        mma_u8(acc[1][j], af[1], b0, b1);
      }
    }
    __syncthreads();                                             // k_term ready
#pragma unroll
    for (int i = 0; i < 2; ++i) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rl = wr + i * 16 + g + 8 * h;
        const int row = q0 + rl;
        if (row >= P.Lq) continue;
        const int rterm = q_term[rl] + kzz;
        float* orow = ob + int64_t(row) * P.ldo;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int cl = wc + j * 8 + 2 * t;
          const int col = k0 + cl;
          if (col >= P.Lk) continue;
          const float v0 = P.scale * float(acc[i][j][2 * h] + rterm + k_term[cl]);
          const float v1 = P.scale * float(acc[i][j][2 * h + 1] + rterm + k_term[cl + 1]);
          if (col + 1 < P.Lk && ((reinterpret_cast<uintptr_t>(orow + col) & 7) == 0)) {
            *reinterpret_cast<float2*>(orow + col) = make_float2(v0, v1);
          } else {
            orow[col] = v0;
            if (col + 1 < P.Lk) orow[col + 1] = v1;
          }
        }
      }
    }
  }
}

}  // namespace

bool scores_supported(const repq_gemm_desc& d) {
  if (d.s_w || d.z_w || d.bias || d.gelu || d.residual || d.acc_debug || d.out_row_sum) return false;
  if (d.out_kind != REPQ_OUT_F32) return false;
  if (d.K > 128 || d.K % 16 != 0) return false;
  const bool both4 = packed4(d.bits_a) && packed4(d.bits_w), both8 = !packed4(d.bits_a) && !packed4(d.bits_w);
  if (!both4 && !both8) return false;
  const int64_t unit = both4 ? 8 : 16;
  auto ok = [&](const uint8_t* p, int64_t ld, int64_t so, int64_t si) {
    return aligned(p, size_t(unit)) && ld % unit == 0 && so % unit == 0 && si % unit == 0;
  };
  if (!ok(d.a_codes, d.lda_bytes, d.a_stride_outer, d.a_stride_inner)) return false;
  if (!ok(d.w_codes, d.ldw_bytes, d.w_stride_outer, d.w_stride_inner)) return false;
  if (int64_t(d.batch_outer) * d.batch_inner > 65535) return false;
  return true;
}

repq_status launch_scores(const repq_gemm_desc& d, cudaStream_t st) {
  ScoresParams P{};
  P.q = d.a_codes; P.k = d.w_codes;
  P.ldq = d.lda_bytes; P.ldk = d.ldw_bytes;
  P.q_so = d.a_stride_outer; P.q_si = d.a_stride_inner; P.k_so = d.w_stride_outer; P.k_si = d.w_stride_inner;
  P.Lq = d.M; P.Lk = d.N; P.dh = d.K; P.dhp = int(round_up(d.K, 32)); P.batch_inner = d.batch_inner;
  P.scale = d.alpha * d.s_a * d.s_w_scalar;
  P.zq = d.z_a; P.zk = d.z_w_scalar;
  P.out = static_cast<float*>(d.out); P.ldo = d.ldo; P.o_so = d.o_stride_outer; P.o_si = d.o_stride_inner;
  P.causal = d.causal;
  dim3 grid((d.M + kTile - 1) / kTile, unsigned(int64_t(d.batch_outer) * d.batch_inner));
  if (packed4(d.bits_a)) scores_kernel<true><<<grid, kThreads, 0, st>>>(P);
  else scores_kernel<false><<<grid, kThreads, 0, st>>>(P);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace repq
