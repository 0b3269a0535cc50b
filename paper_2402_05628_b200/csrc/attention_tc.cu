// Fused attention on integer codes: scores (Eq. 3 with quantized Q and K), Softmax, log-sqrt2 codes (Eq. 15) and
// P.V with the reparameterized log2 de-quantization (Eqs. 16-17) in one kernel.  Scores and codes never leave the
// SM.  The code of a score depends on the row's final Softmax sum, so the keys are walked twice, a visit being 64 keys
// (heads of up to 64 channels) or 128 keys (wider heads):
//   pass 1   S = Q K^T per visit (tcgen05.mma on 8-bit operands into a slot of tensor memory), running row maximum m
//            and sum Z = sum 2^(c (S - m)) (a thread: one row and a quarter of all columns; the four partial results
//            of a row are merged once, after the pass)
//   pass 2   S again, t = 2 (log2 Z + log2 s) - 2 c (S - m), code p = clip(round(t), 0, 2^b - 1), operand values
//            2^(-ceil(p/2)) split by the parity of p into E and O (exact bf16 powers of two), written back as bf16 pairs
//            over the very columns of tensor memory the scores came from; V as exact bf16 integers v - z_v in shared
//            memory; two tcgen05.mma kind::f16 per 16 keys, with the A operand read from tensor memory, accumulate E.V
//            and O.V; O = s s_v (acc_E + sqrt2 acc_O), then the output conversion (Eq. 4 or float)
// Float arithmetic on S is the same as in the separate kernels (float(corr) * (alpha s_q s_k); one ex2 per element
// for Z), so the codes agree with theirs except where the differently ordered sum Z moves a value across a
// rounding tie.
//
// What bounds the kernel is the tensor-core instruction stream and the hand-shakes around it, not the arithmetic: an
// MMA instruction of this size takes about 100 cycles whatever its N, the issuing thread waits for each of its
// barriers in turn, and a worker's visit is a chain of fixed latencies (barrier, tensor-memory load, table look-ups,
// barrier).  Hence:
//  - Warps 0..15 are two groups of eight worker warps that take the visits alternately (group g mod 2 takes visit g;
//    visits are counted over both passes), each with its own slot of tensor memory: while one group waits, the other
//    computes.  Inside a group a thread has one row (its tensor-memory lane) and half of the visit's columns, handled
//    in runs of 16 (one tensor-memory load, arithmetic, in pass 2 one tensor-memory store).
//  - Wide heads use visits of 128 keys (half the instructions per key) and give the P.V MMAs an issuing warp of their
//    own (warp 18), so that the S MMAs (warp 16) are not held up by the wait for the workers' operands.
//  - The E / O operands never touch shared memory, whose bandwidth the V tiles, the table look-ups and the MMAs' B
//    operands already share.
// A group also builds the V tile of its visits (from registers fetched one of its visits ahead) and, for quantizers
// wider than 7 bits, the K tiles of its visits.  Warp 17 (one lane, quantizers of at most 7 bits): K tiles by bulk
// tensor copies.  There the Q tile holds q - z_q as signed bytes and the K tile the raw unsigned codes:
// S' = sum (q - z_q) k differs from the zero-point-corrected sum by -z_k sum (q - z_q), which is the same for every key
// of a row and drops out of the Softmax (maximum and values are taken on S' alone), so no correction and no pass over
// the K bytes is needed.  Under a causal mask, key blocks no row of the CTA may see are skipped.  Every mbarrier wait
// is bounded; when one runs out the kernel records a status code, all roles leave their loops, MMAs in flight are
// drained, tensor memory is freed and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include <cstdlib>

#include "f32x2.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"

namespace repq {
namespace {

using namespace tc;

constexpr int kRows = 128;                  // query rows per CTA (MMA M)
// keys per visit: 64 for heads of up to 64 channels (two CTAs per SM, 256 tensor-memory columns each), 128 for wider
// heads (one CTA per SM): a tensor-core instruction costs about the same time whether it covers 64 or 128 keys
template <int NB> struct VisitKeys { static constexpr int value = NB == 1 ? 64 : 128; };
constexpr int kWorkWarps = 16;                // two groups of eight: 2 per tensor-memory lane quarter and group
constexpr int kGroupWarps = kWorkWarps / 2;
constexpr int kGroupThreads = 32 * kGroupWarps;
constexpr int kParts = kWorkWarps / 4;        // threads that share a row: 2 groups x 2 halves of a block's columns
constexpr int kCols = 16;                     // S columns per tensor-memory load (a run); a thread takes 2 or 4 runs per visit
constexpr int kWorkThreads = 32 * kWorkWarps;
// + S-MMA warp + K-copy warp, and for wide heads a P.V-MMA warp of its own (its waits then do not hold up the S MMAs)
template <int NB> struct Threads { static constexpr int value = kWorkThreads + (NB == 1 ? 64 : 96); };
constexpr uint32_t kQBytes = kRows * 128;         // Q tile: rows of 128 bytes (the head's codes, zero-padded)
constexpr uint32_t kMagicBits = 0x4B400000u;      // float 1.5 * 2^23

struct AttnParams {
  const uint8_t* q; const uint8_t* k; const uint8_t* v;
  int64_t ldq, ldk, ldv, q_so, q_si, k_so, k_si, v_so, v_si;
  int Lq, Lk, dh, batch_inner, causal;
  float scale;            // alpha s_q s_k
  int zq, zk;
  float log2_s;           // log2 of the log-sqrt2 scale
  int qmax_p;             // 2^bits_p - 1
  int z_v, v_small;
  float out_scale;        // s_p s_v
  int out_kind, qmax, pack4;
  float inv_so; int zo;
  void* out; int64_t ldo, o_so, o_si;
  int32_t* out_row_sum;
  int n_pad, tmem_cols, vec_store;
  int no_f8;                                         // keep integer scores where the 8-bit float form would apply
  int pairs, tiles;                                  // (batch, head) pairs and query tiles of 128 rows: the grid is their product
  int32_t* status;
};

// Ring depths.  S: one slot of tensor memory per worker group (2 x 64 or 2 x 128 columns beside the accumulators' 2 x 64
// or 2 x 128).  Heads of up to 64 channels run two CTAs per SM: two K tiles, one V stage.  Wider heads have the SM to
// themselves: four K tiles, two V stages (one per worker group).
template <int NB> struct Rings { static constexpr int kS = 2, kK = NB == 1 ? 2 : 4, kP = NB == 1 ? 1 : 2; };

template <int NB, int kLutBits>
struct AttnShared {
  static constexpr int kS = Rings<NB>::kS, kK = Rings<NB>::kK, kP = Rings<NB>::kP;
  static constexpr int kKeys = VisitKeys<NB>::value;
  static constexpr uint32_t kKBytes = kKeys * 128;
  static constexpr uint32_t kVBlockBytes = kKeys * 128;       // the visit's keys x 64 channels of bf16
  alignas(1024) uint8_t q[kQBytes];
  alignas(1024) uint8_t k[kK][kKBytes];
  alignas(1024) uint8_t v[kP][NB * kVBlockBytes];
  int row_term[kRows];                              // -z_k qsum[m] + d_h z_q z_k
  int col_term[4][kKeys];                           // -z_q ksum[n], ring of 4 visits
  float stat_m[kParts][kRows], stat_z[kParts][kRows];   // pass-1 results of the column parts of every row
  static constexpr int kLutEntries = kLutBits ? (1 << kLutBits) + 1 : 1;
  uint32_t lut[kLutEntries][32];                    // table-driven codes: [code][lane] = E value | O value << 16 (one bank per
                                                    // lane); the last entry repeats the top code (a clamp at 2^bits that
                                                    // rounds up lands there)
  alignas(8) uint64_t k_full[kK];
  uint64_t k_empty[kK];                             // K tile read by its S MMAs (bulk-copy variant)
  uint64_t s_full[kS], s_empty[kS], s_spent[kS], p_full[kP], p_empty[kP];   // s_empty: read in pass 1; s_spent: P.V MMAs of a
                                                                            // pass-2 visit have read the operands written over S
  uint64_t stats_ready, acc_full, done, done_pv;
  uint32_t tmem_base;
  volatile int abort;
};

__device__ __forceinline__ uint32_t tile_offset(int row, int piece) {
  return uint32_t(row >> 3) * 1024u + uint32_t(row & 7) * 128u + (uint32_t(piece ^ (row & 7)) << 4);
}
__device__ __forceinline__ int sum_bytes(const uint4& v) {
  return __dp4a(v.x, 0x01010101u, __dp4a(v.y, 0x01010101u, __dp4a(v.z, 0x01010101u, __dp4a(v.w, 0x01010101u, 0u))));
}
// Bytewise c - z (two's complement) for codes and zero points below 128: with the top bit of every byte of c set
// no borrow crosses a byte, and flipping that bit back leaves c - z mod 256.
__device__ __forceinline__ uint32_t sub_bytes(uint32_t c, uint32_t z4) { return ((c | 0x80808080u) - z4) ^ 0x80808080u; }
__device__ __forceinline__ uint4 sub_bytes(const uint4& c, uint32_t z4) {
  return make_uint4(sub_bytes(c.x, z4), sub_bytes(c.y, z4), sub_bytes(c.z, z4), sub_bytes(c.w, z4));
}
// Bytes in two's complement (within [-127, 127]) -> sign bit and magnitude.
__device__ __forceinline__ uint32_t sign_magnitude(uint32_t x) { return __vabs4(x) | (x & 0x80808080u); }
__device__ __forceinline__ uint4 sign_magnitude(const uint4& c) {
  return make_uint4(sign_magnitude(c.x), sign_magnitude(c.y), sign_magnitude(c.z), sign_magnitude(c.w));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// NB: 64-channel blocks of the head; kLutBits: width of the Softmax codes when their operand values come from the
// per-lane table (4, 6, or 8 where one CTA per SM leaves room for 257 entries), 0: integer arithmetic
// kMode: how the scores are formed.
//   kCorrected  unsigned Q and K tiles, accumulators corrected by the row and column zero-point terms
//   kCentred    q - z_q fits a signed byte (quantizers of at most 7 bits): the Q tile holds q - z_q, the K tile the raw
//               codes, the S MMAs run signed x unsigned and their accumulators need no correction
//   kCentredF8  4-bit quantizers (|q - z_q| <= 15, k <= 15): the same tiles read as 8-bit floats.  A byte below 16 is
//               the e4m3 number byte * 2^-9 (subnormals and the first binade are linear in the byte), so the raw K codes
//               are already such numbers and the Q tile stores sign and magnitude of q - z_q.  Products and sums are
//               multiples of 2^-18 below 2^-3, exact in the float32 accumulator, which therefore holds
//               2^-18 sum (q - z_q) k as a float: the int -> float conversion of every score is gone (the factor 2^18 is
//               folded into the score scale on the host, exactly)
enum : int { kCorrected = 0, kCentred = 1, kCentredF8 = 2 };
template <int NB, int kLutBits, int kMode>
__global__ void __launch_bounds__(Threads<NB>::value, NB == 1 ? 2 : 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_k, AttnParams P) {
  using Shared = AttnShared<NB, kLutBits>;
  constexpr int kKeys = Shared::kKeys;
  constexpr uint32_t kKBytes = Shared::kKBytes, kVBlockBytes = Shared::kVBlockBytes;
  constexpr bool kSplitIssue = NB != 1;                   // P.V MMAs issued by a warp of their own
  constexpr int kRuns = kKeys / (2 * kCols);              // runs of 16 columns per thread and visit
  constexpr bool kLut = kLutBits != 0;
  constexpr bool kCentered = kMode != kCorrected;
  constexpr bool kF8 = kMode == kCentredF8;
  constexpr int kS = Shared::kS, kK = Shared::kK, kP = Shared::kP;      // ring depths (powers of two)
  constexpr int kAccCol = kS * kKeys;                     // first tensor-memory column of the P.V accumulators
  auto ring = [](int i, int depth) { return i & (depth - 1); };
  auto lap = [](int i, int depth) { return uint32_t(i / depth) & 1u; };       // parity of the slot's use count
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Shared& S = *reinterpret_cast<Shared*>(smem_raw);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Under a causal mask the later a query tile, the more key blocks it visits: the CTAs run longest first (every
  // pair's last tile, then every pair's tile before it, ...), so that the tail of the grid is made of the short ones
  // (measured: -6 % on 2048-token causal rows).  Without a mask the tiles of a pair stay neighbours (the tile-major
  // order measured 2 % slower there).
  int pair, tile;
  if (P.causal) {
    const int slot = int(blockIdx.x) / P.pairs;
    pair = int(blockIdx.x) - slot * P.pairs;
    tile = P.tiles - 1 - slot;
  } else {
    pair = int(blockIdx.x) / P.tiles;
    tile = int(blockIdx.x) - pair * P.tiles;
  }
  const int bo = pair / P.batch_inner, bi = pair % P.batch_inner;
  const int q0 = tile * kRows;
  const int shift = P.Lk - P.Lq;
  const int k_end = P.causal ? max(1, min(P.Lk, min(q0 + kRows, P.Lq) + shift)) : P.Lk;
  const int min_valid = P.causal ? max(0, min(P.Lk, q0 + 1 + shift)) : P.Lk;   // fewest keys any row of the CTA sees
  const int nb = (k_end + kKeys - 1) / kKeys;             // key blocks of a visit's size; every one is visited in both passes
  const int ksteps = (P.dh + 31) >> 5;                    // S MMAs of K = 32 per key block
  const int pieces = P.dh >> 4;                           // 16-byte pieces of a Q / K row

  if (tid == 0) {
    for (int s = 0; s < kK; ++s) {
      mbar_init(smem_u32(&S.k_full[s]), kCentered ? 1 : kGroupWarps);
      mbar_init(smem_u32(&S.k_empty[s]), 1);
    }
    for (int s = 0; s < kS; ++s) {
      mbar_init(smem_u32(&S.s_full[s]), 1);
      mbar_init(smem_u32(&S.s_empty[s]), kGroupWarps);
      mbar_init(smem_u32(&S.s_spent[s]), 1);
    }
    for (int s = 0; s < kP; ++s) {
      mbar_init(smem_u32(&S.p_full[s]), kGroupWarps);
      mbar_init(smem_u32(&S.p_empty[s]), 1);
    }
    mbar_init(smem_u32(&S.stats_ready), kWorkWarps);
    mbar_init(smem_u32(&S.acc_full), 1);
    mbar_init(smem_u32(&S.done), 1);
    mbar_init(smem_u32(&S.done_pv), 1);
    S.abort = 0;
    if (smem_u32(smem_raw) & 1023u) {                     // the swizzled tiles need this alignment
      atomicCAS(P.status, 0, 49);
      S.abort = 1;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWorkWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&S.tmem_base)), "r"(uint32_t(P.tmem_cols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  // everything above touched no global memory of the kernel chain
  grid_dependency_wait();
  grid_dependency_trigger();

  // The first K tiles are asked for before the Q tile is staged (their barriers must be visible first), so that the
  // copies' latency and the Q loads' run side by side.
  int k_issued = 0;
  if (kCentered) {
    __syncthreads();
    if (warp == kWorkWarps + 1 && lane == 0) {
      for (; k_issued < kK && k_issued < 2 * nb; ++k_issued) {
        const uint32_t bar = smem_u32(&S.k_full[k_issued]);
        mbar_expect_tx(bar, kKBytes);
        tma_load_3d(smem_u32(S.k[k_issued]), &map_k, bar, bi * int(P.k_si), (k_issued < nb ? k_issued : k_issued - nb) * kKeys, bo);
      }
    }
  }

  // ---- K rows (quantizers wider than 7 bits): a group stages the K tiles of its own visits, 8 threads per key with one
  // 16-byte piece each, two keys per thread; Q rows: 4 threads per row, 2 pieces each
  const uint8_t* k_base = P.k + bo * P.k_so + bi * P.k_si;
  const int gt = tid & (kGroupThreads - 1);       // thread in group
  const int kkey = gt >> 3, kq = gt & 7;          // keys kkey, kkey + 32, ... of a visit
  constexpr int kKeysPerThread = kKeys / 32;
  uint4 kreg[kKeysPerThread];                                  // the thread's pieces of the K tile its group stages next
  auto fetch_k = [&](int block) {
#pragma unroll
    for (int u = 0; u < kKeysPerThread; ++u) {
      kreg[u] = make_uint4(0u, 0u, 0u, 0u);
      const int key = block * kKeys + kkey + 32 * u;
      if (key < P.Lk && kq < pieces) kreg[u] = __ldg(reinterpret_cast<const uint4*>(k_base + int64_t(key) * P.ldk) + kq);
    }
  };
  const uint32_t zq4 = uint32_t(P.zq) * 0x01010101u;
  // K tile and column terms of visit g from kreg; then the pieces of the group's visit after that are requested
  auto stage_k = [&](int g) {
    uint8_t* tile = S.k[ring(g, kK)];
#pragma unroll
    for (int u = 0; u < kKeysPerThread; ++u) {
      if (kq < 2 * ksteps) *reinterpret_cast<uint4*>(tile + tile_offset(kkey + 32 * u, kq)) = kreg[u];
      int sum = sum_bytes(kreg[u]);
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sum += __shfl_xor_sync(0xffffffffu, sum, 4);
      if (kq == 0) S.col_term[g & 3][kkey + 32 * u] = -P.zq * sum;
    }
    fence_async_smem();
    __syncwarp();
    if ((tid & 31) == 0) mbar_arrive(smem_u32(&S.k_full[ring(g, kK)]));
    if (g + 2 < 2 * nb) fetch_k(g + 2 < nb ? g + 2 : g + 2 - nb);
  };

  if (warp < kWorkWarps) {
    if (!kCentered && (tid >> 8) < 2 * nb) fetch_k((tid >> 8) < nb ? (tid >> 8) : (tid >> 8) - nb);   // the group's first visit
    const uint8_t* q_base = P.q + bo * P.q_so + bi * P.q_si;
    const int qrow = (tid >> 2) & (kRows - 1), qh = tid & 3;
    int s = 0;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int piece = 2 * qh + j;
      uint4 w = make_uint4(0u, 0u, 0u, 0u);
      if (q0 + qrow < P.Lq && piece < pieces) {
        w = __ldg(reinterpret_cast<const uint4*>(q_base + int64_t(q0 + qrow) * P.ldq) + piece);
        if (kCentered) w = sub_bytes(w, zq4);
        if (kF8) w = sign_magnitude(w);
      }
      if (piece < 2 * ksteps) *reinterpret_cast<uint4*>(S.q + tile_offset(qrow, piece)) = w;
      s += sum_bytes(w);
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (qh == 0) S.row_term[qrow] = -P.zk * s + P.dh * P.zq * P.zk;
    if (kLut) {
      for (int i = tid; i < Shared::kLutEntries * 32; i += kWorkThreads) {
        const uint32_t code = min(uint32_t(i >> 5), uint32_t(Shared::kLutEntries - 2)), kk = (code + 1u) >> 1;
        const uint32_t bits16 = kk > 126u ? 0u : (127u - kk) << 7;   // bf16 bits of 2^-ceil(code/2) (0 below the normal range)
        S.lut[0][i] = (code & 1u) ? bits16 << 16 : bits16;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S.tmem_base;
  volatile int* abort = &S.abort;

  // P.V: D = f32, A = B = bf16, A from tensor memory, B MN-major, N = n_pad, M = 128
  const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (uint32_t(P.n_pad >> 3) << 17) |
                            (uint32_t(kRows >> 4) << 24);
  // P.V MMAs of block j, from the operands the workers of visit nb + j left: A in tensor memory, in the columns of
  // S(nb + j) (a row's E values of keys 16 s .. 16 s + 15 in the 8 columns from 16 s, its O values in the next 8),
  // B = the V tile in shared memory
  auto issue_pv = [&](int j) {
    const int pb = ring(j, kP);
    if (!mbar_wait(smem_u32(&S.p_full[pb]), lap(j, kP), abort, 43, P.status)) return false;
    tc_fence_after();
    const uint64_t dv = smem_desc_sw128(smem_u32(S.v[pb]), kVBlockBytes);
    const int keys_here = min(kKeys, k_end - j * kKeys);
    const int steps = (keys_here + 15) >> 4;                       // 16 keys per MMA
    const uint32_t a_base = tmem_base + uint32_t(ring(nb + j, kS) * kKeys);
    for (int s = 0; s < steps; ++s) {
      const uint32_t accumulate = (j | s) != 0 ? 1u : 0u;
      const uint32_t a_e = a_base + uint32_t(16 * s);
      umma_f16_ts(tmem_base + uint32_t(kAccCol), a_e, dv + uint64_t(128 * s), idesc_pv, accumulate);
      umma_f16_ts(tmem_base + uint32_t(kAccCol + P.n_pad), a_e + 8u, dv + uint64_t(128 * s), idesc_pv, accumulate);
    }
    umma_commit(smem_u32(&S.s_spent[ring(nb + j, kS)]));
    umma_commit(smem_u32(&S.p_empty[pb]));
    return true;
  };

  if (warp == kWorkWarps) {
    // ---------------------------------------------------------------- MMA issue
    if (lane == 0) {
      // S: D = s32, A = B = unsigned 8-bit, both K-major, N = 64, M = 128
      // (operand formats: 0 = unsigned, 1 = signed bytes)
      // kCentredF8: D = f32, A = B = e4m3 (format 0)
      constexpr uint32_t idesc_s = kF8 ? (1u << 4) | (uint32_t(kKeys >> 3) << 17) | (uint32_t(kRows >> 4) << 24)
                                       : (2u << 4) | (uint32_t(kCentered) << 7) | (0u << 10) | (uint32_t(kKeys >> 3) << 17) |
                                             (uint32_t(kRows >> 4) << 24);
      const uint64_t dq = smem_desc_sw128(smem_u32(S.q));
      bool ok = true;
      auto issue_s = [&](int g) {                          // S of key block g % nb, g counted over both passes
        const int b = ring(g, kS), kb = ring(g, kK);
        if (!mbar_wait(smem_u32(&S.k_full[kb]), lap(g, kK), abort, 41, P.status)) return false;
        // the slot's last user: a pass-1 visit (the workers have read it) or a pass-2 visit (its P.V MMAs have read
        // the operands the workers wrote over it)
        const int prev = g - kS;
        if (prev >= nb) {
          const int first = nb + ((b - nb) & (kS - 1));         // the slot's first pass-2 visit
          if (!mbar_wait(smem_u32(&S.s_spent[b]), lap(prev - first, kS), abort, 42, P.status)) return false;
        } else if (prev >= 0) {
          if (!mbar_wait(smem_u32(&S.s_empty[b]), lap(prev, kS), abort, 42, P.status)) return false;
        }
        tc_fence_after();
        const uint64_t dk = smem_desc_sw128(smem_u32(S.k[kb]));
        for (int s = 0; s < ksteps; ++s) {
          if (kF8) umma_f8(tmem_base + uint32_t(b * kKeys), dq + uint64_t(2 * s), dk + uint64_t(2 * s), idesc_s, s != 0 ? 1u : 0u);
          else umma_i8(tmem_base + uint32_t(b * kKeys), dq + uint64_t(2 * s), dk + uint64_t(2 * s), idesc_s, s != 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&S.s_full[b]));
        if (kCentered) umma_commit(smem_u32(&S.k_empty[kb]));     // the K tile may be refilled once these MMAs have read it
        return true;
      };
      if (kSplitIssue) {
        // this thread issues the S MMAs only; each waits for its K tile and for its slot
        for (int g = 0; g < 2 * nb && ok && !*abort; ++g) ok = issue_s(g);
      } else {
        // one thread for both: the S MMAs stay one visit ahead of the P.V MMAs
        int next_s = 0;
        for (; next_s < nb + 1 && next_s < 2 * nb && ok && !*abort; ++next_s) ok = issue_s(next_s);
        for (int j = 0; j < nb && ok && !*abort; ++j) {
          if (next_s < 2 * nb) {
            if (!issue_s(next_s)) { ok = false; break; }
            ++next_s;
          }
          ok = issue_pv(j);
        }
        if (ok && !*abort) umma_commit(smem_u32(&S.acc_full));
      }
      umma_commit(smem_u32(&S.done));
      mbar_drain(smem_u32(&S.done), 0);
    }
  } else if (kSplitIssue && warp == kWorkWarps + 2) {
    // ---------------------------------------------------------------- P.V MMA issue (wide heads)
    if (lane == 0) {
      bool ok = true;
      for (int j = 0; j < nb && ok && !*abort; ++j) ok = issue_pv(j);
      if (ok && !*abort) umma_commit(smem_u32(&S.acc_full));
      umma_commit(smem_u32(&S.done_pv));
      mbar_drain(smem_u32(&S.done_pv), 0);
    }
  } else if (warp == kWorkWarps + 1) {
    // ---------------------------------------------------------------- K tiles by bulk tensor copies
    if (kCentered && lane == 0) {
      int issued = k_issued;
      for (int g = k_issued; g < 2 * nb && !*abort; ++g) {
        const int b = ring(g, kK);
        if (!mbar_wait(smem_u32(&S.k_empty[b]), lap(g, kK) ^ 1u, abort, 48, P.status)) break;
        const uint32_t bar = smem_u32(&S.k_full[b]);
        mbar_expect_tx(bar, kKBytes);
        // box: 128 bytes of the head's row (bytes past d_h meet zero bytes of the Q tile), 64 keys (rows past Lk are
        // zero-filled), one batch item
        tma_load_3d(smem_u32(S.k[b]), &map_k, bar, bi * int(P.k_si), (g < nb ? g : g - nb) * kKeys, bo);
        ++issued;
      }
      // the copies issued last must have landed before this CTA may exit
      for (int i = issued > kK ? issued - kK : 0; i < issued; ++i) mbar_drain(smem_u32(&S.k_full[ring(i, kK)]), lap(i, kK));
    }
  } else {
    // ---------------------------------------------------------------- tiles, Softmax arithmetic, epilogue
    const int quarter = warp & 3, half = (warp >> 2) & 1, group = warp >> 3;
    const int part = group * 2 + half;                    // which of the four threads of a row this one is
    const int r = quarter * 32 + lane;                    // the thread's row inside the CTA = its tensor-memory lane
    const int row = q0 + r;
    const int valid = row < P.Lq ? (P.causal ? max(1, min(P.Lk, row + 1 + shift)) : P.Lk) : 0;   // keys the row sees
    const int my_row_term = S.row_term[r];
    // a warp whose 32 rows all lie past Lq (the tail of the last query tile) skips the code arithmetic of pass 2 and
    // writes zero operands; it still stages K and V and arrives on every barrier
    const bool dead_warp = __all_sync(0xffffffffu, valid == 0);
    const float c = 1.4426950408889634f;
    const float k1 = -2.f * c;
    const float qs = float(P.qmax_p + 1), inv_qs = 1.f / qs;      // 2^bits and its reciprocal (exact)
    const uint32_t u_top = kMagicBits + uint32_t(P.qmax_p);
    const float magic = __uint_as_float(kMagicBits);
    const uint32_t taddr_s = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(half * kRuns * kCols);

    // V items of a visit: the group's 256 threads take the visit's keys x 8 NB groups of 8 channels in kVItems steps;
    // a thread keeps its channel group and moves down the keys (32 / NB keys per step, a multiple of the swizzle period)
    constexpr int kVKeyStep = 32 / NB;
    constexpr int kVItems = kKeys / kVKeyStep;
    const int v_g8 = gt % (8 * NB), v_key0 = gt / (8 * NB);
    const bool v_chan_live = v_g8 * 8 < P.dh;
    const uint8_t* v_ptr = P.v + bo * P.v_so + bi * P.v_si + int64_t(v_key0) * P.ldv + v_g8 * 8;
    const uint32_t v_off = uint32_t(v_g8 >> 3) * kVBlockBytes + tile_offset(v_key0, v_g8 & 7);
    uint2 vraw[kVItems];
    auto fetch_v = [&](int block) {
#pragma unroll
      for (int qi = 0; qi < kVItems; ++qi) {
        vraw[qi] = make_uint2(0u, 0u);
        const int key = block * kKeys + v_key0 + qi * kVKeyStep;
        if (block < nb && v_chan_live && key < P.Lk)
          vraw[qi] = __ldg(reinterpret_cast<const uint2*>(v_ptr + int64_t(block * kKeys + qi * kVKeyStep) * P.ldv));
      }
    };
    const float vz = __uint_as_float(kMagicBits) + float(P.z_v);
    const __nv_bfloat162 vz2 = __float2bfloat162_rn(128.f + float(P.z_v));

    float m = -CUDART_INF_F, z = 0.f;       // pass 1: running maximum and sum of this thread's columns
    float k0 = 0.f;                         // pass 2: 2 (log2 Z + log2 s), with m the row's final maximum

    // Start of a visit: the S MMAs of visit g have completed.  (Where the group stages its own K tiles, the tile of its
    // next visit is written here: with a ring of two it is the tile those MMAs have just finished reading.)
    auto begin_visit = [&](int g) -> bool {
      if (!mbar_wait(smem_u32(&S.s_full[ring(g, kS)]), lap(g, kS), abort, 44, P.status)) return false;
      tc_fence_after();
      if (!kCentered && g + 2 < 2 * nb) stage_k(g + 2);
      return true;
    };
    // Run h (16 columns) of the thread's scores of visit g in units of the score scale, as floats: the accumulator
    // itself (kCentredF8), the converted accumulator (kCentred), or the converted corr = acc - z_k qsum - z_q ksum +
    // d_h z_q z_k (kCorrected).  The buffer is handed back after the second run.  Keys the row may not see are dealt
    // with by the callers, in the runs that reach past the keys the thread's row sees: the values themselves are left
    // as they come from tensor memory, so that the common path carries no selects or copies.
    auto read_run = [&](int g, int h, float (&sf)[kCols]) {
      uint32_t rn[kCols];
      __syncwarp();
      tmem_ld16(taddr_s + uint32_t(ring(g, kS) * kKeys + h * kCols), rn);
      tmem_ld_wait();
      if (h == kRuns - 1 && g < nb) {               // pass 1: the slot is free; pass 2: the operands go back into it
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&S.s_empty[ring(g, kS)]));
      }
      if (kF8) {
#pragma unroll
        for (int e = 0; e < kCols; ++e) sf[e] = __uint_as_float(rn[e]);
      } else if (kCentered) {
#pragma unroll
        for (int e = 0; e < kCols; ++e) sf[e] = float(int32_t(rn[e]));
      } else {
        const int* ct = S.col_term[g & 3] + (half * kRuns + h) * kCols;
#pragma unroll
        for (int e4 = 0; e4 < kCols / 4; ++e4) {
          const int4 c4 = *reinterpret_cast<const int4*>(ct + 4 * e4);
          sf[4 * e4 + 0] = float(int32_t(rn[4 * e4 + 0]) + my_row_term + c4.x);
          sf[4 * e4 + 1] = float(int32_t(rn[4 * e4 + 1]) + my_row_term + c4.y);
          sf[4 * e4 + 2] = float(int32_t(rn[4 * e4 + 2]) + my_row_term + c4.z);
          sf[4 * e4 + 3] = float(int32_t(rn[4 * e4 + 3]) + my_row_term + c4.w);
        }
      }
    };

    // ---- pass 1: running maximum and sum of one run.  The maximum is taken on the unscaled values (S = scale * sf is
    // monotonic in sf); a key the row may not see contributes nothing (`seen`: columns e < seen are keys the row sees).
    // Exponents and sums on packed pairs.
    auto stats_run = [&](const float (&sf)[kCols], int seen) {
      const float sc = P.scale * c;                             // exponent of 2 per unit of sf
      if (__builtin_expect(seen >= kCols, 1)) {
        float bm = max3(sf[0], sf[1], sf[2]);
#pragma unroll
        for (int e = 3; e + 1 < kCols; e += 2) bm = max3(bm, sf[e], sf[e + 1]);
        bm = fmaxf(bm, sf[kCols - 1]);
        const float mn = fmaxf(m, P.scale * bm);
        const f32x2 sc2 = splat2(sc), nm2 = splat2(-(mn * c));
        f32x2 acc = 0ull;                                       // even columns in the low lane, odd ones in the high lane
#pragma unroll
        for (int e = 0; e < kCols; e += 2) {
          float a0, a1;
          unpack2(fma2(pack2(sf[e], sf[e + 1]), sc2, nm2), a0, a1);
          acc = add2(acc, pack2(ex2(a0), ex2(a1)));
        }
        float acc0, acc1;
        unpack2(acc, acc0, acc1);
        z = z * ex2((m - mn) * c) + (acc0 + acc1);     // m = -inf at first: factor 0
        m = mn;
      } else if (seen > 0) {
        float bm = sf[0];
#pragma unroll
        for (int e = 1; e < kCols; ++e)
          if (e < seen) bm = fmaxf(bm, sf[e]);
        const float mn = fmaxf(m, P.scale * bm);
        const float mnc = mn * c;
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < kCols; ++e)
          if (e < seen) acc += ex2(fmaf(sf[e], sc, -mnc));
        z = z * ex2((m - mn) * c) + acc;
        m = mn;
      }
    };

    // ---- pass 2: codes and operand values of one run.
    // Eq. 15: p = clip(round(t), 0, qmax), t = k0 - 2 c (S - m); rounding half to even by the float add of
    // 1.5 * 2^23, which leaves p in the low mantissa bits u - kMagicBits.  The pair (E, O) of bf16 operand values,
    // 2^-ceil(p/2) on the side of p's parity and 0 on the other, comes from a per-lane table for 4-bit codes and
    // from integer arithmetic for wider ones.  A masked key gets (0, 0).
    const uint32_t lut_addr = smem_u32(&S.lut[0][lane]) - (kMagicBits << 7);
    auto code_run = [&](const float (&sf)[kCols], int seen, uint32_t (&eow)[kCols]) {
      // a warp none of whose rows sees a key of the run (the block past the last key, the blocks beyond the diagonal
      // under a causal mask) writes zero operands without any arithmetic
      if (dead_warp || !__any_sync(0xffffffffu, seen > 0)) {
#pragma unroll
        for (int e = 0; e < kCols; ++e) eow[e] = 0u;
        return;
      }
      uint32_t eo[kCols];
      // S - m on packed pairs; then t 2^-bits out of one saturating fma each (k1 and k0 scaled by 2^-bits, exact, so the
      // value is t rounded as before and clamped to [0, 1] whatever the inputs: rows past Lq carry m = -inf, Z = 0), and
      // the scaling back and the rounding as one more packed fma
      constexpr float kSteps = kLut ? float(1 << kLutBits) : 0.f;
      const float steps = kLut ? kSteps : qs, inv_steps = kLut ? 1.f / kSteps : inv_qs;
      const float k1s = k1 * inv_steps, k0s = k0 * inv_steps;
      const f32x2 scale2 = splat2(P.scale), nm2 = splat2(-m), steps2 = splat2(steps), magic2 = splat2(magic);
#pragma unroll
      for (int e = 0; e < kCols; e += 2) {
        float x0, x1, w0, w1;
        unpack2(fma2(pack2(sf[e], sf[e + 1]), scale2, nm2), x0, x1);
        asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(w0) : "f"(x0), "f"(k1s), "f"(k0s));
        asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(w1) : "f"(x1), "f"(k1s), "f"(k0s));
        float uf[2];
        unpack2(fma2(pack2(w0, w1), steps2, magic2), uf[0], uf[1]);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (kLut) {
            // table-driven codes; 2^bits (t within half a code of it) reads the table's copy of the top entry
            asm("ld.shared.u32 %0, [%1];" : "=r"(eo[e + h]) : "r"(lut_addr + (__float_as_uint(uf[h]) << 7)));
          } else {
            // wider codes: the top code by one integer minimum
            const uint32_t u = min(__float_as_uint(uf[h]), u_top);
            const int kk = int((u - kMagicBits + 1u) >> 1);                       // ceil(p / 2)
            const uint32_t val = uint32_t(max(127 - kk, 0)) << 7;                 // bf16 bits of 2^-kk (0 below the normal range)
            eo[e + h] = (u & 1u) ? val << 16 : val;
          }
        }
      }
      if (__builtin_expect(seen < kCols, 0)) {
#pragma unroll
        for (int e = 0; e < kCols; ++e)
          if (e >= seen) eo[e] = 0u;
      }
      // E pairs (even key in the low half) in words 0..7, O pairs in words 8..15
#pragma unroll
      for (int e = 0; e < kCols / 2; ++e) {
        eow[e] = __byte_perm(eo[2 * e], eo[2 * e + 1], 0x5410);
        eow[kCols / 2 + e] = __byte_perm(eo[2 * e], eo[2 * e + 1], 0x7632);
      }
    };

    bool ok = true;
    if (!kCentered && group < 2 * nb) stage_k(group);          // the K tile of the group's first visit
    // ---- pass 1 over the group's visits
    for (int g = group; g < nb && !*abort; g += 2) {
      if (!begin_visit(g)) { ok = false; break; }
      const int seen = valid - (g * kKeys + half * kRuns * kCols);   // of the thread's columns
#pragma unroll
      for (int h = 0; h < kRuns; ++h) {
        float sf[kCols];
        read_run(g, h, sf);
        stats_run(sf, seen - h * kCols);
      }
    }
    // merge the four column parts of every row: m = max, Z = sum of the rescaled partial sums (same order in every
    // thread of the row, so that all of them hold the same Z)
    if (ok && !*abort) {
      S.stat_m[part][r] = m;
      S.stat_z[part][r] = z;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.stats_ready));
      ok = mbar_wait(smem_u32(&S.stats_ready), 0, abort, 45, P.status);
    }
    const int g2 = nb + ((nb ^ group) & 1);                     // the group's first visit of pass 2
    if (ok && !*abort) {
      float mn = -CUDART_INF_F;
#pragma unroll
      for (int q = 0; q < kParts; ++q) mn = fmaxf(mn, S.stat_m[q][r]);
      float zt = 0.f;
#pragma unroll
      for (int q = 0; q < kParts; ++q) {
        const float mq = S.stat_m[q][r];
        if (mq > -CUDART_INF_F) zt += S.stat_z[q][r] * ex2((mq - mn) * c);
      }
      m = mn;
      k0 = 2.f * (log2f(zt) + P.log2_s);
      fetch_v(g2 - nb);
    }
    // ---- pass 2 over the group's visits
    for (int g = g2; g < 2 * nb && ok && !*abort; g += 2) {
      const int j = g - nb;
      if (!begin_visit(g)) { ok = false; break; }
      const int seen = valid - (j * kKeys + half * kRuns * kCols);
      // E and O operands of a run: bf16 pairs written back over the run's own 16 columns of S(g) (8 columns of E, then 8
      // of O), from where the P.V MMAs take their A operand; nothing else reads those columns any more
#pragma unroll
      for (int h = 0; h < kRuns; ++h) {
        float sf[kCols];
        read_run(g, h, sf);
        uint32_t eow[kCols];
        code_run(sf, seen - h * kCols, eow);
        __syncwarp();
        tmem_st16(taddr_s + uint32_t(ring(g, kS) * kKeys + h * kCols), eow);
      }
      // the stage of the V tile: the MMAs of the block that used it before must have read it
      const int pb = ring(j, kP);
      if (!mbar_wait(smem_u32(&S.p_empty[pb]), lap(j, kP) ^ 1u, abort, 46, P.status)) { ok = false; break; }
#pragma unroll
      for (int qi = 0; qi < kVItems; ++qi) {
        uint32_t o4[4] = {0u, 0u, 0u, 0u};
        if (v_chan_live && j * kKeys + v_key0 + qi * kVKeyStep < P.Lk) {
          const uint32_t b03 = vraw[qi].x, b47 = vraw[qi].y;
          if (P.v_small) {
            // v - z_v as bf16: for codes below 128, 128 + v is the bit pattern 0x4300 | v and the bf16 subtraction exact
            const uint32_t w[4] = {__byte_perm(b03, 0x43434343u, 0x4140), __byte_perm(b03, 0x43434343u, 0x4342),
                                   __byte_perm(b47, 0x43434343u, 0x4140), __byte_perm(b47, 0x43434343u, 0x4342)};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 hh = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&w[e]), vz2);
              o4[e] = *reinterpret_cast<const uint32_t*>(&hh);
            }
          } else {
            float f[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              f[e] = __uint_as_float(__byte_perm(b03, kMagicBits, 0x7650 + e)) - vz;
              f[4 + e] = __uint_as_float(__byte_perm(b47, kMagicBits, 0x7650 + e)) - vz;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 hh = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
              o4[e] = *reinterpret_cast<const uint32_t*>(&hh);
            }
          }
        }
        *reinterpret_cast<uint4*>(S.v[pb] + v_off + uint32_t(qi * (kVKeyStep / 8)) * 1024u) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
      }
      fetch_v(j + 2);
      fence_async_smem();
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.p_full[pb]));
    }

    // ---------------------------------------------------------------- epilogue: one row per thread, the 16-column
    // chunks of the accumulators dealt to the four warps of a lane quarter
    if (ok && !*abort && mbar_wait(smem_u32(&S.acc_full), 0, abort, 47, P.status)) {
      tc_fence_after();
      const float kSqrt2 = 1.41421356237309504880f;
      const float zo_lo = float(-P.zo), zo_hi = float(P.qmax - P.zo);
      const bool row_ok = row < P.Lq;
      const int64_t roff = bo * P.o_so + bi * P.o_si + int64_t(row) * P.ldo;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(kAccCol);
      int code_sum = 0;
      for (int c0 = part * 16; c0 < P.dh; c0 += kParts * 16) {      // the 16-column chunks of the accumulators, dealt to the parts
        uint32_t re[16], ro[16];
        __syncwarp();
        tmem_ld16(taddr + uint32_t(c0), re);
        tmem_ld16(taddr + uint32_t(P.n_pad + c0), ro);
        tmem_ld_wait();
        float v[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = P.out_scale * fmaf(kSqrt2, __uint_as_float(ro[e]), __uint_as_float(re[e]));
        if (!row_ok) continue;
        if (P.out_kind == REPQ_OUT_F32) {
          float* o = static_cast<float*>(P.out) + roff + c0;
          if (P.vec_store) {
#pragma unroll
            for (int e = 0; e < 4; ++e) reinterpret_cast<float4*>(o)[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = v[e];
          }
        } else if (P.out_kind == REPQ_OUT_BF16) {
          __nv_bfloat16* o = static_cast<__nv_bfloat16*>(P.out) + roff + c0;
          if (P.vec_store) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
              w[e] = *reinterpret_cast<const uint32_t*>(&h);
            }
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
            if (P.vec_store) *reinterpret_cast<uint2*>(orow + (c0 >> 1)) = make_uint2(w0, w1);
            else {
#pragma unroll
              for (int e = 0; e < 4; ++e) { orow[(c0 >> 1) + e] = uint8_t(w0 >> (8 * e)); orow[(c0 >> 1) + 4 + e] = uint8_t(w1 >> (8 * e)); }
            }
          } else {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w[e] = q[4 * e] | (q[4 * e + 1] << 8) | (q[4 * e + 2] << 16) | (q[4 * e + 3] << 24);
            if (P.vec_store) *reinterpret_cast<uint4*>(orow + c0) = make_uint4(w[0], w[1], w[2], w[3]);
            else {
#pragma unroll
              for (int e = 0; e < 16; ++e) orow[c0 + e] = uint8_t(q[e]);
            }
          }
        }
      }
      if (P.out_row_sum != nullptr && P.out_kind == REPQ_OUT_CODES && row_ok && part * 16 < P.dh)
        atomicAdd(P.out_row_sum + int64_t(bo) * P.Lq + row, code_sum);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (warp < kWorkWarps) tmem_st_wait();          // an error path may leave a tensor-memory store in flight
  tc_fence_before();
  __syncthreads();
  if (warp == kWorkWarps) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(P.tmem_cols)) : "memory");
  }
}

// Tensor map of the K codes for the bulk-copy variant: (bytes of a row, keys, batch items); a box is 128 bytes x the keys of a visit.
repq_status make_k_map(CUtensorMap* map, const AttnParams& P, int batch_outer, int keys) {
  EncodeTiledFn fn = encode_fn();
  REPQ_REQUIRE(fn != nullptr, REPQ_CUDA_ERROR, "attention: cuTensorMapEncodeTiled is not available");
  const cuuint64_t span = cuuint64_t(P.batch_inner - 1) * cuuint64_t(P.k_si) + cuuint64_t(P.dh);    // bytes the heads cover
  const cuuint64_t dims[3] = {span, cuuint64_t(P.Lk), cuuint64_t(batch_outer)};
  const cuuint64_t strides[2] = {cuuint64_t(P.ldk), cuuint64_t(P.k_so)};
  const cuuint32_t box[3] = {128, cuuint32_t(keys), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t*>(P.k), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  REPQ_REQUIRE(r == CUDA_SUCCESS, REPQ_CUDA_ERROR, "attention: K tensor map failed with code %d", int(r));
  return REPQ_OK;
}

template <int NB, int kLutBits, int kMode>
repq_status launch_kernel(const AttnParams& P, int64_t pairs, cudaStream_t st) {
  const size_t smem = sizeof(AttnShared<NB, kLutBits>);
  REPQ_CUDA(cudaFuncSetAttribute(attention_tc_kernel<NB, kLutBits, kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  AttnParams Q = P;
  Q.pairs = int(pairs);
  Q.tiles = (P.Lq + kRows - 1) / kRows;
  if (kMode == kCentredF8) Q.scale = P.scale * 262144.f;      // the accumulators hold 2^-18 sum (q - z_q) k
  CUtensorMap map_k{};
  if (kMode != kCorrected) REPQ_TRY(make_k_map(&map_k, P, int(pairs / P.batch_inner), VisitKeys<NB>::value));
  dim3 grid(unsigned(Q.tiles) * unsigned(pairs));
  REPQ_CUDA(launch_chained(attention_tc_kernel<NB, kLutBits, kMode>, grid, dim3(Threads<NB>::value), smem, st, map_k, Q));
  note_launch();
  return REPQ_OK;
}

template <int NB, int kLutBits>
repq_status launch(const AttnParams& P, int64_t pairs, int qmax_qk, cudaStream_t st) {
  // q - z_q and k - z_k as signed bytes: codes and zero points below 128 and differences within [-128, 127]
  // (the K tiles of this variant come by bulk tensor copies: row and batch strides must be usable as tensor-map strides)
  const bool centred = qmax_qk < 128 && P.zq >= 0 && P.zq < 128 && P.zk >= 0 && P.zk < 128 && P.k_so > 0 &&
                       P.ldk < (int64_t(1) << 40) && P.k_so < (int64_t(1) << 40) &&
                       int64_t(P.batch_inner - 1) * P.k_si + P.dh <= P.ldk;
  // 4-bit quantizers with the zero point of Q inside the code range: the tiles are also valid 8-bit floats
  const bool f8 = centred && qmax_qk <= 15 && P.zq <= 15 && !P.no_f8;
  if (f8) return launch_kernel<NB, kLutBits, kCentredF8>(P, pairs, st);
  return centred ? launch_kernel<NB, kLutBits, kCentred>(P, pairs, st) : launch_kernel<NB, kLutBits, kCorrected>(P, pairs, st);
}

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_attention(const repq_attention_desc* d, void* stream) {
  REPQ_REQUIRE(d, REPQ_INVALID_ARG, "attention: NULL descriptor");
  REPQ_REQUIRE(d->batch_outer > 0 && d->batch_inner > 0 && d->Lq >= 0 && d->Lk > 0 && d->d_h > 0, REPQ_INVALID_ARG, "attention: bad sizes");
  if (d->Lq == 0) return REPQ_OK;
  REPQ_REQUIRE(d->q_codes && d->k_codes && d->v_codes && d->out, REPQ_INVALID_ARG, "attention: NULL pointer");
  REPQ_REQUIRE(bits_ok(d->bits_qkv) && bits_ok(d->bits_p), REPQ_INVALID_ARG, "attention: bits must be 4, 6 or 8");
  REPQ_REQUIRE(!packed4(d->bits_qkv), REPQ_UNSUPPORTED, "attention: Q, K, V codes must be stored one per byte (REPQ_BYTE_CODES)");
  REPQ_REQUIRE(d->d_h % 16 == 0 && d->d_h <= 128, REPQ_UNSUPPORTED, "attention: d_h = %d must be a multiple of 16, at most 128", d->d_h);
  REPQ_REQUIRE(d->s_q > 0.f && d->s_k > 0.f && d->s_v > 0.f && d->s_p > 0.f && d->alpha > 0.f, REPQ_INVALID_ARG, "attention: scales must be positive");
  REPQ_REQUIRE(!d->causal || d->Lk >= d->Lq, REPQ_INVALID_ARG, "attention: causal needs Lk >= Lq");
  auto rows16 = [](const void* p, int64_t ld, int64_t so, int64_t si) { return aligned(p, 16) && ld % 16 == 0 && so % 16 == 0 && si % 16 == 0; };
  REPQ_REQUIRE(rows16(d->q_codes, d->ldq_bytes, d->q_stride_outer, d->q_stride_inner) &&
               rows16(d->k_codes, d->ldk_bytes, d->k_stride_outer, d->k_stride_inner), REPQ_ALIGNMENT,
               "attention: Q and K rows must be 16-byte aligned");
  REPQ_REQUIRE(aligned(d->v_codes, 8) && d->ldv_bytes % 8 == 0 && d->v_stride_outer % 8 == 0 && d->v_stride_inner % 8 == 0, REPQ_ALIGNMENT,
               "attention: V rows must be 8-byte aligned");
  REPQ_REQUIRE(d->ldq_bytes >= d->d_h && d->ldk_bytes >= d->d_h && d->ldv_bytes >= d->d_h, REPQ_INVALID_ARG, "attention: row stride shorter than d_h");
  const int qmax_v = code_max(d->bits_qkv);
  REPQ_REQUIRE(d->z_v >= qmax_v - 256 && d->z_v <= 256, REPQ_UNSUPPORTED, "attention: z_v = %d puts v - z_v outside [-256, 256]", d->z_v);
  REPQ_REQUIRE(d->out_kind == REPQ_OUT_F32 || d->out_kind == REPQ_OUT_BF16 || d->out_kind == REPQ_OUT_CODES, REPQ_INVALID_ARG, "attention: unknown out_kind");
  const int64_t esz = d->out_kind == REPQ_OUT_F32 ? 4 : d->out_kind == REPQ_OUT_BF16 ? 2 : 1;
  REPQ_REQUIRE(aligned(d->out, size_t(esz)), REPQ_ALIGNMENT, "attention: out is not element-aligned");
  const int64_t pairs = int64_t(d->batch_outer) * d->batch_inner;
  REPQ_REQUIRE(pairs <= 65535, REPQ_UNSUPPORTED, "attention: more than 65535 (batch, head) pairs");
  AttnParams P{};
  P.q = d->q_codes; P.k = d->k_codes; P.v = d->v_codes;
  P.ldq = d->ldq_bytes; P.ldk = d->ldk_bytes; P.ldv = d->ldv_bytes;
  P.q_so = d->q_stride_outer; P.q_si = d->q_stride_inner; P.k_so = d->k_stride_outer; P.k_si = d->k_stride_inner;
  P.v_so = d->v_stride_outer; P.v_si = d->v_stride_inner;
  P.Lq = d->Lq; P.Lk = d->Lk; P.dh = d->d_h; P.batch_inner = d->batch_inner; P.causal = d->causal;
  P.scale = d->alpha * d->s_q * d->s_k;
  P.zq = d->z_q; P.zk = d->z_k;
  P.log2_s = log2f(d->s_p);
  P.qmax_p = code_max(d->bits_p);
  P.z_v = d->z_v;
  P.v_small = qmax_v < 128 && d->z_v > -128 && d->z_v < 128;
  P.out_scale = d->s_p * d->s_v;
  P.out_kind = d->out_kind;
  if (d->out_kind == REPQ_OUT_CODES) {
    REPQ_REQUIRE(bits_ok(d->out_bits) && d->out_scale > 0.f, REPQ_INVALID_ARG, "attention: bad output quantizer");
    REPQ_REQUIRE(d->out_zero > -(1 << 20) && d->out_zero < (1 << 20), REPQ_INVALID_ARG, "attention: |out_zero| must be below 2^20");
    P.qmax = code_max(d->out_bits); P.pack4 = packed4(d->out_bits); P.inv_so = 1.f / d->out_scale; P.zo = d->out_zero;
  }
  P.out = d->out; P.ldo = d->ldo; P.o_so = d->o_stride_outer; P.o_si = d->o_stride_inner;
  P.out_row_sum = d->out_kind == REPQ_OUT_CODES ? d->out_row_sum : nullptr;
  P.n_pad = (d->d_h + 15) / 16 * 16;
  P.tmem_cols = d->d_h <= 64 ? 256 : 512;      // 2 x 64 + 2 x 64, or 4 x 64 + 2 x 128 columns
  const int64_t chunk_bytes = d->out_kind == REPQ_OUT_CODES && packed4(d->out_bits) ? 8 : 16 * esz;
  const int64_t al = chunk_bytes < 16 ? chunk_bytes : 16;
  P.vec_store = aligned(d->out, size_t(al)) && (d->ldo * esz) % al == 0 && (d->o_stride_outer * esz) % al == 0 &&
                (d->o_stride_inner * esz) % al == 0;
  P.status = device_status_word();
  REPQ_REQUIRE(P.status != nullptr, REPQ_CUDA_ERROR, "attention: device status word unavailable");
  {
    // read at every call, so that a test can compare the two score forms in one process
    const char* e = getenv("REPQ_ATTENTION_INT_SCORES");
    P.no_f8 = e && *e && *e != '0';
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the per-lane table of the Softmax codes' operand values: 17 / 65 entries everywhere; the 257 entries of 8-bit codes
  // (33 KB) only where the head already limits the SM to one CTA
  if (d->d_h <= 64) {
    if (P.qmax_p <= 15) return launch<1, 4>(P, pairs, qmax_v, st);
    if (P.qmax_p <= 63) return launch<1, 6>(P, pairs, qmax_v, st);
    return launch<1, 0>(P, pairs, qmax_v, st);
  }
  if (P.qmax_p <= 15) return launch<2, 4>(P, pairs, qmax_v, st);
  if (P.qmax_p <= 63) return launch<2, 6>(P, pairs, qmax_v, st);
  return launch<2, 8>(P, pairs, qmax_v, st);
}
