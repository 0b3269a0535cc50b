// Integer GEMM on the 5th-generation tensor cores: TMA-fed shared-memory operand ring, single-thread
// tcgen05.mma (kind::i8, u8 x u8 -> s32) into tensor memory, and an epilogue that reads the int32
// accumulators back with tcgen05.ld and applies the zero-point correction, scale, bias, GELU, residual
// and re-quantization of the quantized linear layer.
//
// One persistent CTA per SM; roles by warp:
//   warp 0       TMA producer (one elected lane): A tile 128 x 128 B, W tile BN x 128 B per stage, 128-byte
//                swizzle, zero fill outside the matrices
//   warp 1       tensor-memory allocation and MMA issue (one elected lane): 4 MMAs of K = 32 per stage,
//                accumulators double-buffered in TMEM (2 x 256 columns) so the epilogue of tile i overlaps
//                the main loop of tile i + 1
//   warps 2..17  epilogue: warp w reads TMEM lanes 32 (w mod 4) .. +31 (one output row per thread) and a
//                64-column slice of the accumulator columns
//   packed weights (4-bit, two codes per byte; 6-bit, four codes in three bytes): 12 epilogue warps (tiles of at most
//                192 columns) and 4 converter warps.  The weight tile arrives packed and the converters expand it into
//                the 128-byte-swizzled byte tile the MMA descriptor expects (there is no 4- or 6-bit integer MMA); one
//                more barrier hop between the copy and the MMA, weights stay packed in HBM
// The tile width BN (256, 192 or 128) is chosen per problem: rounds of tiles over the SMs times a per-round time
// with a fixed part.  Packed 4-bit activations are expanded to one code per byte by a separate pass into the
// workspace (inside the block the producers write byte codes, so that pass does not run there).
//
// For short K the epilogue, not the tensor pipe, sets the pace (K = 768: 3072 tensor-pipe cycles per
// 128 x 256 tile against 32768 outputs), so it is written for few instructions per output and few waits per
// tile: every epilogue warp stages the per-column terms of its own 64 columns in its own shared-memory buffer
// (no barrier between warps) from plain loads issued one tile ahead and reads them as vectors, the output
// quantizer is folded into them where nothing sits between the GEMM and the re-quantization, rounding uses
// the float adder (add 1.5 * 2^23), byte codes of at most 7 bits are clamped by one saturating fma instead of
// comparisons, and a bf16 residual comes in either by row-per-lane loads requested before the accumulator is
// waited for or, for short K, by bulk tensor copies (one 32 x 64 box per epilogue warp, one tile ahead).
//
// Every wait on an mbarrier is bounded: when it runs out the kernel records a status code, all roles
// leave their loops, in-flight copies and MMAs are drained, tensor memory is freed and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>

#include "kernels.h"
#include "tc_ptx.cuh"

namespace repq {
namespace {

constexpr int BM = 128, BK = 128;                   // BK in bytes (= codes); BN is a template parameter
constexpr int kMaxBN = 256;
constexpr int kChunk = 16;                           // accumulator columns per tcgen05.ld / per store
constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;                      // TMEM columns between the two accumulator buffers
constexpr int kSliceCols = 64;                       // accumulator columns per epilogue warp
constexpr int kSliceChunks = kSliceCols / kChunk;
constexpr int kConvWarps = 4;                        // converter warps of the packed-weight variant, which gives up four
constexpr int kConvThreads = 32 * kConvWarps;        // epilogue warps for them (same CTA size, same register budget)
constexpr int kEpiWarpsW4 = kEpiWarps - kConvWarps;
constexpr int kMaxBNW4 = kEpiWarpsW4 / 4 * kSliceCols;   // 192: one 64-column slice per epilogue warp of a lane quarter
constexpr uint32_t kABytes = BM * BK;
constexpr uint32_t kMagicBits = 0x4B400000u;         // 1.5 * 2^23

__device__ int32_t g_status_word = 0;

struct alignas(16) ColTerms {                          // per output column of a warp's slice, staged once per tile
  int32_t nzw[kSliceCols];  // -z_w[j]
  int32_t kw[kSliceCols];   // -z_a * wsum[j]
  float sc[kSliceCols];     // alpha s_a s_w[j]   (times 1/s_o in direct re-quantization mode)
  float bi[kSliceCols];     // bias[j]            (times 1/s_o in direct re-quantization mode)
};

constexpr uint32_t kResBytes = 32 * 128;            // bf16 residual of one warp and tile: 32 rows x 64 columns

// RES (bf16 output with a bf16 residual, tiles of at most 192 columns): the residual of a tile comes in by bulk tensor
// copies, one 32 x 64 box per epilogue warp, asked for one tile ahead; the output values are written over the residual
// values they were computed from and the box leaves by one bulk tensor store (no staging buffer beside it)
// WP: 0 = weight tiles arrive as bytes; 4 / 6 = packed (64 / 96 bytes per row of 128 codes), expanded by the converters
template <int BN, bool RES, int WP>
struct SharedStorage {
  static constexpr bool W4 = WP != 0;               // (any packed form)
  // kStages: ring of the bulk copies (activation tile + weight tile as it arrives).  kStagesB: ring of byte weight
  // tiles the MMA reads: the same ring when the weights arrive as bytes; with packed weights a short ring of its own
  // (the hop from converter to MMA is short), which leaves room for a deeper copy ring ahead of the converters.
  static constexpr int kStages = WP == 6 ? 4 : WP == 4 ? 5 : 4;
  static constexpr int kPackedRow = BK * (WP ? WP : 8) / 8;        // bytes of a packed tile row
  static constexpr int kStagesB = W4 ? 2 : kStages;
  static constexpr int kEpi = W4 ? kEpiWarpsW4 : kEpiWarps;
  alignas(1024) uint8_t a[kStages][kABytes];
  alignas(1024) uint8_t b[kStagesB][BN * BK];
  alignas(1024) uint8_t res[RES ? (BN / kSliceCols) * 4 * kResBytes : 1024];   // one box per active epilogue warp
  uint64_t res_full[kEpiWarps];
  alignas(1024) uint8_t epi[RES ? 1 : kEpi][1024]; // per-warp staging box of the epilogue's bulk stores (RES: the residual box itself)
  ColTerms cols[kEpi];                            // each epilogue warp stages the terms of its own slice: no barrier
  alignas(128) uint8_t bp[W4 ? kStages : 1][W4 ? BN * kPackedRow : 128];   // packed weight tiles: unswizzled rows
  alignas(8) uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t ready[kStagesB];                         // packed variant: byte weight tile written by the converters
  uint64_t bfree[kStagesB];                         //                 ... and read by the MMAs
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t done;
  uint32_t tmem_base;
  volatile int abort;
};

static_assert(sizeof(SharedStorage<kMaxBN, false, 0>) <= 227 * 1024 && sizeof(SharedStorage<kMaxBNW4, false, 4>) <= 227 * 1024 &&
              sizeof(SharedStorage<kMaxBNW4, false, 6>) <= 227 * 1024 && sizeof(SharedStorage<192, true, 0>) <= 227 * 1024,
              "shared storage exceeds the 227 KB a CTA may use");

using namespace tc;

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, int code) {
  return tc::mbar_wait(bar, parity, abort, code, &g_status_word);
}

// Shared-memory matrix descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) { return smem_desc_sw128(addr); }

// Instruction descriptor: D = s32, A = B = unsigned 8-bit, both K-major, N = bn, M = 128.
constexpr uint32_t idesc_for(int bn) {
  return (2u << 4) | (0u << 7) | (0u << 10) | (uint32_t(bn >> 3) << 17) | (uint32_t(BM >> 4) << 24);
}

// Order of the output tiles.  The row tiles are cut into panels of P.panel; a panel is walked column tile by column
// tile with its row tiles innermost.  The CTAs that run at the same time then share a panel of activations small
// enough to stay in L2 while the weight tiles stream past it (with long K the activations of all row tiles do not
// fit, and walking every row tile per column tile read them from DRAM once per wave of CTAs).
// Every role of the CTA needs the origin of every tile it visits, and a division by a run-time number is a chain of
// some 25 dependent instructions that all epilogue warps would walk through at the same moment; the divisors are
// fixed per launch, so the host supplies their reciprocals (n / d = umulhi(n, ceil(2^32 / d)) while n d < 2^32).
struct FastDiv { uint32_t d, mul; };                            // mul == 0: plain division
inline FastDiv fast_div(uint32_t d, uint64_t n_max) {
  FastDiv f{d, 0u};
  if (d > 1 && n_max * d < (uint64_t(1) << 32)) f.mul = uint32_t((uint64_t(1) << 32) / d) + 1u;
  return f;
}
__device__ __forceinline__ uint32_t div_by(uint32_t n, const FastDiv& f) { return f.mul ? __umulhi(n, f.mul) : n / f.d; }
struct TileOrder {
  int full;                    // tiles inside whole panels
  int panel, last_rows;        // row tiles of a whole panel and of the last, shorter one
  int m_tiles;
  FastDiv by_panel_tiles;      // panel * n_tiles
  FastDiv by_panel, by_last_rows;
};
struct TileOrigin { int m0, n0; };
__device__ __forceinline__ TileOrigin tile_origin(int tile, const TileOrder& T, int bn) {
  uint32_t rows = uint32_t(T.panel), first = 0, t = uint32_t(tile);
  uint32_t col;
  if (tile >= T.full) {                                          // the last, shorter panel
    t = uint32_t(tile - T.full);
    rows = uint32_t(T.last_rows);
    first = uint32_t(T.m_tiles) - rows;
    col = div_by(t, T.by_last_rows);
  } else {
    const uint32_t p = div_by(t, T.by_panel_tiles);
    first = p * uint32_t(T.panel);
    t -= p * T.by_panel_tiles.d;
    col = div_by(t, T.by_panel);
  }
  return TileOrigin{int(first + (t - col * rows)) * BM, int(col) * bn};
}

struct TcParams {
  int M, N, K;
  const int32_t* asum;
  const int32_t* wsum;
  int direct_requant;          // codes out, no GELU, no residual: 1/s_o is folded into the column terms
  int w_packed4;               // weight tiles arrive packed (4: two codes per byte, 6: four in three bytes) and are
                               // expanded in shared memory; 0: byte tiles
  TileOrder order;             // panels of row tiles (see TileOrder)
  EpilogueParams ep;
};

enum : int { kOutF32 = 0, kOutBf16 = 1, kOutC4 = 2, kOutC8 = 3 };   // compile-time output kinds of the fast path

// Output quantizer of one 16-column chunk (Eq. 4 with the chunk's column group).
struct ChunkQuant {
  float mult, lo, hi;
  uint32_t pack_k;     // 4-bit: sum_e (magic_bits - z_o) << 4e
  uint32_t z4;         // 8-bit: z_o replicated in every byte
  int zo;
  float inv_qs, qs, csat;   // byte codes of at most 7 bits: 1 / 2^bits, 2^bits, (z_o - magic) / 2^bits
  int qs_shift;             //   bits
};

__device__ __forceinline__ ChunkQuant chunk_quant(const EpilogueParams& ep, const TcParams& P, int col0) {
  const int gw = ep.group_width;
  const int group = (col0 >= gw) + (col0 >= 2 * gw) + (col0 >= 3 * gw);
  // (selects, not run-time indexing: an indexed kernel parameter makes every thread keep a copy of the parameters in
  // local memory)
  const int zo = group == 0 ? ep.out_zero[0] : group == 1 ? ep.out_zero[1] : group == 2 ? ep.out_zero[2] : ep.out_zero[3];
  const float inv = group == 0 ? ep.inv_out_scale[0] : group == 1 ? ep.inv_out_scale[1] : group == 2 ? ep.inv_out_scale[2] : ep.inv_out_scale[3];
  ChunkQuant q;
  q.mult = P.direct_requant ? 1.f : inv;
  q.lo = float(-zo);
  q.hi = float(ep.qmax - zo);
  q.pack_k = (kMagicBits - uint32_t(zo)) * 0x11111111u;
  q.z4 = (uint32_t(zo) & 0xFFu) * 0x01010101u;
  q.zo = zo;
  q.qs_shift = 32 - __clz(ep.qmax);                      // qmax = 2^bits - 1
  q.qs = __uint_as_float(uint32_t(127 + q.qs_shift) << 23);         // 2^bits
  q.inv_qs = __uint_as_float(uint32_t(127 - q.qs_shift) << 23);     // 2^-bits
  q.csat = (float(zo) - __uint_as_float(kMagicBits)) * q.inv_qs;    // exact: an integer below 2^24 times a power of two
  return q;
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}

// The warp's 1 KB staging buffer holds a box of 32 rows x 32 bytes in the 32-byte swizzle of the output tensor
// map (16-byte slot j of row r sits at r * 32 + ((j ^ ((r >> 2) & 1)) << 4): conflict-free for one row per lane).
// begin: the previous bulk store must have finished reading the buffer; end: make the generic-proxy writes
// visible to the bulk-copy engine, then one lane issues the store (rows / columns outside the matrix are clipped).
__device__ __forceinline__ void box_begin(int lane) {
  if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  __syncwarp();
}
__device__ __forceinline__ void box_end(const CUtensorMap* map, uint32_t buf, int lane, int x, int y) {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  if (lane == 0) {
    tma_store_2d(map, buf, x, y);
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }
}
__device__ __forceinline__ uint32_t box_slot(uint32_t buf, int lane, int j) {
  return buf + uint32_t(lane) * 32u + (uint32_t(j ^ ((lane >> 2) & 1)) << 4);
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float fma_sat(float a, float b, float c) {       // fma clamped to [0, 1]
  float d;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void sts64(uint32_t addr, uint32_t a, uint32_t b) {
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(a), "r"(b) : "memory");
}

// Fast path: chunk c (16 columns) of the warp's 64-column slice, one row per lane, output kind fixed at compile
// time.  Values go to the staging buffer and leave through bulk tensor stores: one per chunk (bf16), two per
// chunk (f32), one per two chunks (byte codes) or one per slice (4-bit codes).
template <int OUT>
__device__ __forceinline__ void emit_chunk(const CUtensorMap* map_out, uint32_t buf, int lane, const ChunkQuant& q,
                                           float (&v)[kChunk], int c, int col0, int row0, int& code_sum, bool direct, bool sat) {
  if constexpr (OUT == kOutF32) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      box_begin(lane);
#pragma unroll
      for (int j = 0; j < 2; ++j)
        sts128(box_slot(buf, lane, j), __float_as_uint(v[8 * h + 4 * j]), __float_as_uint(v[8 * h + 4 * j + 1]),
               __float_as_uint(v[8 * h + 4 * j + 2]), __float_as_uint(v[8 * h + 4 * j + 3]));
      box_end(map_out, buf, lane, col0 + 8 * h, row0);
    }
  } else if constexpr (OUT == kOutBf16) {
    uint32_t w[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
      w[k] = *reinterpret_cast<const uint32_t*>(&h);
    }
    box_begin(lane);
    sts128(box_slot(buf, lane, 0), w[0], w[1], w[2], w[3]);
    sts128(box_slot(buf, lane, 1), w[4], w[5], w[6], w[7]);
    box_end(map_out, buf, lane, col0, row0);
  } else {
    const float magic = __uint_as_float(kMagicBits);
    uint32_t u[kChunk];
    if (OUT == kOutC8 && sat) {
      // Byte codes of at most 7 bits, no comparisons: r = magic + round_half_even(t) by the float adder (one fma
      // from the value when the scale is still to be applied), w = clamp((r - magic + z_o) / 2^bits, 0, 1) by a
      // saturating fma whose unclamped result is exact, u = magic + 2^bits w.  The low byte of u is the code,
      // except that 2^bits stands for the top code 2^bits - 1; that bit is subtracted after packing.
      uint32_t w[4];
      // (the adds and multiply-adds around the saturating one on packed pairs: same operations, same bits)
      const f32x2 magic2 = splat2(magic), qs2 = splat2(q.qs), mult2 = splat2(q.mult);
#pragma unroll
      for (int e = 0; e < kChunk; e += 2) {
        float r0, r1, u0, u1;
        const f32x2 v2 = pack2(v[e], v[e + 1]);
        unpack2(direct ? add2(v2, magic2) : fma2(v2, mult2, magic2), r0, r1);
        unpack2(fma2(pack2(fma_sat(r0, q.inv_qs, q.csat), fma_sat(r1, q.inv_qs, q.csat)), qs2, magic2), u0, u1);
        u[e] = __float_as_uint(u0);
        u[e + 1] = __float_as_uint(u1);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t p = __byte_perm(__byte_perm(u[4 * i], u[4 * i + 1], 0x0040), __byte_perm(u[4 * i + 2], u[4 * i + 3], 0x0040), 0x5410);
        w[i] = p - ((p >> q.qs_shift) & 0x01010101u);
        code_sum += __dp4a(w[i], 0x01010101u, 0u);
      }
      if ((c & 1) == 0) box_begin(lane);
      sts128(box_slot(buf, lane, c & 1), w[0], w[1], w[2], w[3]);
      if (c & 1) box_end(map_out, buf, lane, col0 - kChunk, row0);
      return;
    }
    {
      const f32x2 magic2 = splat2(magic), mult2 = splat2(q.mult);
#pragma unroll
      for (int e = 0; e < kChunk; e += 2) {
        float t0, t1, u0, u1;
        unpack2(mul2(pack2(v[e], v[e + 1]), mult2), t0, t1);
        unpack2(add2(pack2(fminf(fmaxf(t0, q.lo), q.hi), fminf(fmaxf(t1, q.lo), q.hi)), magic2), u0, u1);   // magic_bits + round_half_even(t)
        u[e] = __float_as_uint(u0);
        u[e + 1] = __float_as_uint(u1);
      }
    }
    if constexpr (OUT == kOutC4) {
      uint32_t w[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        w[i] = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) w[i] += u[i * 8 + e] << (4 * e);
        w[i] -= q.pack_k;
        code_sum += __dp4a(w[i] & 0x0F0F0F0Fu, 0x01010101u, 0u) + __dp4a((w[i] >> 4) & 0x0F0F0F0Fu, 0x01010101u, 0u);
      }
      if (c == 0) box_begin(lane);
      sts64(box_slot(buf, lane, c >> 1) + uint32_t(c & 1) * 8u, w[0], w[1]);     // 8 bytes = 16 codes
      if (c == kSliceChunks - 1) box_end(map_out, buf, lane, (col0 - (kSliceChunks - 1) * kChunk) >> 1, row0);
    } else {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        w[i] = __vadd4(__byte_perm(__byte_perm(u[4 * i], u[4 * i + 1], 0x0040), __byte_perm(u[4 * i + 2], u[4 * i + 3], 0x0040), 0x5410), q.z4);
        code_sum += __dp4a(w[i], 0x01010101u, 0u);
      }
      if ((c & 1) == 0) box_begin(lane);
      sts128(box_slot(buf, lane, c & 1), w[0], w[1], w[2], w[3]);
      if (c & 1) box_end(map_out, buf, lane, col0 - kChunk, row0);
    }
  }
}

// General path for one chunk of one thread (ragged rows / columns, float32 residual, accumulator dump):
// element by element, kept out of line so that the common path stays small.
__device__ __noinline__ void slow_chunk(const EpilogueParams& ep, const TcParams& P, const ColTerms& C, const uint32_t* r,
                                        int cl, int64_t m, int col0, int32_t asum_c, int* code_sum) {
  const ChunkQuant q = chunk_quant(ep, P, col0);
  const float magic = __uint_as_float(kMagicBits);
  auto code_of = [&](float v) {
    const float t = fminf(fmaxf(v * q.mult, q.lo), q.hi);
    return (__float_as_uint(t + magic) - kMagicBits) + uint32_t(q.zo);
  };
  for (int e = 0; e < kChunk; e += 2) {                // column pairs (the chunk starts at an even column)
    const int j = col0 + e;
    if (j >= P.N) break;
    const bool two = j + 1 < P.N;
    float v[2] = {0.f, 0.f};
    for (int h = 0; h < (two ? 2 : 1); ++h) {
      if (ep.acc_debug) ep.acc_debug[m * P.N + j + h] = int32_t(r[e + h]);
      float x = fmaf(C.sc[cl + e + h], float(int32_t(r[e + h]) + C.nzw[cl + e + h] * asum_c + C.kw[cl + e + h]), C.bi[cl + e + h]);
      if (ep.gelu) x = gelu_erf(x);
      if (ep.residual) {
        const int64_t off = m * ep.ld_residual + j + h;
        x += ep.residual_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(ep.residual)[off])
                              : static_cast<const float*>(ep.residual)[off];
      }
      v[h] = x;
    }
    if (ep.rope != nullptr && j < ep.rope_cols)
      rope_rotate(ep.rope[int64_t(m % ep.rope_period) * (ep.rope_dim >> 1) + ((j % ep.rope_dim) >> 1)], v[0], v[1]);
    if (ep.glu) {
      const float hv = silu_mul(v[0], v[1]);
      const int oc = j >> 1;
      if (ep.out_kind == REPQ_OUT_F32) {
        static_cast<float*>(ep.out)[m * ep.ldo + oc] = hv;
      } else if (ep.out_kind == REPQ_OUT_BF16) {
        static_cast<__nv_bfloat16*>(ep.out)[m * ep.ldo + oc] = __float2bfloat16_rn(hv);
      } else {
        const uint32_t code = code_of(hv);
        *code_sum += int(code);
        static_cast<uint8_t*>(ep.out)[m * ep.ldo + oc] = uint8_t(code);
      }
      continue;
    }
    if (ep.out_kind == REPQ_OUT_F32) {
      float* o = static_cast<float*>(ep.out) + m * ep.ldo + j;
      o[0] = v[0];
      if (two) o[1] = v[1];
    } else if (ep.out_kind == REPQ_OUT_BF16) {
      __nv_bfloat16* o = static_cast<__nv_bfloat16*>(ep.out) + m * ep.ldo + j;
      o[0] = __float2bfloat16_rn(v[0]);
      if (two) o[1] = __float2bfloat16_rn(v[1]);
    } else {
      const uint32_t c0 = code_of(v[0]), c1 = two ? code_of(v[1]) : 0u;
      *code_sum += int(c0 + c1);
      uint8_t* orow = static_cast<uint8_t*>(ep.out) + m * ep.ldo;
      if (ep.pack4) {
        orow[j >> 1] = uint8_t(c0 | (c1 << 4));
      } else {
        orow[j] = uint8_t(c0);
        if (two) orow[j + 1] = uint8_t(c1);
      }
    }
  }
}

// PAIR: step on neighbouring column pairs ahead of the output conversion, compiled into the common epilogue only
// where asked for: kPairNone, kPairRope (rotary embedding), kPairGlu (gated product; byte codes out)
enum : int { kPairNone = 0, kPairRope = 1, kPairGlu = 2 };

template <int BN, int OUT, bool RES, int PAIR, int WP>
__global__ void __launch_bounds__(kThreads, 1)
qgemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_res, const __grid_constant__ TcParams P) {
  using Storage = SharedStorage<BN, RES, WP>;
  constexpr bool W4 = WP != 0;                           // weights arrive packed
  constexpr int kStages = Storage::kStages;
  constexpr int EW = W4 ? kEpiWarpsW4 : kEpiWarps;       // epilogue warps of this variant
  static_assert(!W4 || BN <= kMaxBNW4, "the packed-weight variant has three column slices");
  constexpr uint32_t kBBytes = BN * BK;
  constexpr uint32_t kIdesc = idesc_for(BN);
  // 1024-byte alignment (swizzle atoms) is requested from the declaration so that the compiler keeps
  // treating every access below as a shared-memory access (a hand-aligned generic pointer would not)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Storage& S = *reinterpret_cast<Storage*>(smem_raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (P.M + BM - 1) / BM, n_tiles = (P.N + BN - 1) / BN;
  const int tiles = m_tiles * n_tiles;
  const int kblocks = (P.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&S.full[s]), 1);
      mbar_init(smem_u32(&S.empty[s]), 1);
    }
    for (int s = 0; s < Storage::kStagesB; ++s) { mbar_init(smem_u32(&S.ready[s]), kConvWarps); mbar_init(smem_u32(&S.bfree[s]), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&S.tmem_full[a]), 1); mbar_init(smem_u32(&S.tmem_empty[a]), EW); }
    for (int w = 0; w < kEpiWarps; ++w) mbar_init(smem_u32(&S.res_full[w]), 1);
    mbar_init(smem_u32(&S.done), 1);
    S.abort = 0;
    if (smem_u32(smem_raw) & 1023u) {              // the swizzled tiles need the alignment asked for above
      atomicCAS(&g_status_word, 0, 9);
      S.abort = 1;
    }
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
  // everything above touched no global memory of the kernel chain
  grid_dependency_wait();
  grid_dependency_trigger();

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      long long issued = 0;
      for (int tile = blockIdx.x; tile < tiles && !*abort; tile += gridDim.x) {
        const TileOrigin o = tile_origin(tile, P.order, BN);
        const int m0 = o.m0, n0 = o.n0;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(smem_u32(&S.empty[stage]), phase ^ 1, abort, 1)) break;
          const uint32_t bar = smem_u32(&S.full[stage]);
          mbar_expect_tx(bar, kABytes + (W4 ? uint32_t(BN * Storage::kPackedRow) : kBBytes));
          tma_load_2d(smem_u32(S.a[stage]), &map_a, bar, kb * BK, m0);
          if constexpr (W4) tma_load_2d(smem_u32(S.bp[stage]), &map_b, bar, kb * Storage::kPackedRow, n0);
          else tma_load_2d(smem_u32(S.b[stage]), &map_b, bar, kb * BK, n0);
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
      uint32_t stage = 0, phase = 0, bstage = 0, bphase = 0;
      int it = 0;
      for (int tile = blockIdx.x; tile < tiles && !*abort; tile += gridDim.x, ++it) {
        const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
        if (!mbar_wait(smem_u32(&S.tmem_empty[acc]), acc_phase ^ 1, abort, 2)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        bool ok = true;
        for (int kb = 0; kb < kblocks; ++kb) {
          // packed weights: the converters hand over a byte tile (they have waited for the copies themselves, so the
          // activation tile of the same k-block has landed as well)
          if (!mbar_wait(smem_u32(W4 ? &S.ready[bstage] : &S.full[stage]), W4 ? bphase : phase, abort, 3)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = smem_desc(smem_u32(S.a[stage])), db = smem_desc(smem_u32(S.b[W4 ? bstage : stage]));
#pragma unroll
          for (int k = 0; k < BK / 32; ++k)
            umma_i8(d_tmem, da + uint64_t(k * 2), db + uint64_t(k * 2), kIdesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(smem_u32(&S.empty[stage]));          // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1; }
          if constexpr (W4) {
            umma_commit(smem_u32(&S.bfree[bstage]));       // and the byte tile for the converters
            if (++bstage == Storage::kStagesB) { bstage = 0; bphase ^= 1; }
          }
        }
        if (!ok) break;
        umma_commit(smem_u32(&S.tmem_full[acc]));           // accumulator complete
      }
      // all MMAs issued by this thread must have completed before tensor memory is freed
      umma_commit(smem_u32(&S.done));
      const long long t0 = clock64();
      while (!mbar_try_wait(smem_u32(&S.done), 0) && clock64() - t0 < kWaitCycles) {}
    }
  } else if (W4 && warp >= 2 + EW) {
    // ---------------------------------------------------------------- converters (packed 4-bit weights)
    // A packed tile holds BN rows of 64 bytes (128 codes, even index in the low nibble).  Thread ct takes 16-byte
    // pieces ct, ct + 128, ...: piece g = (row g / 4, codes 32 (g % 4) ..) becomes the two 16-byte pieces 2 (g % 4) and
    // 2 (g % 4) + 1 of the row's 128 bytes, stored where the 128-byte swizzle puts them.  Reads are consecutive
    // across the warp; the stores of eight neighbouring threads cover two rows and all eight swizzled positions.
    const int ct = int(threadIdx.x) - 32 * (2 + EW);
    uint32_t stage = 0, phase = 0, bstage = 0, bphase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok && !*abort; tile += gridDim.x) {
      for (int kb = 0; kb < kblocks; ++kb) {
        // the packed tile has landed, and the MMAs that read the byte tile's previous content have completed
        if (!mbar_wait(smem_u32(&S.full[stage]), phase, abort, 7)) { ok = false; break; }
        if (!mbar_wait(smem_u32(&S.bfree[bstage]), bphase ^ 1, abort, 8)) { ok = false; break; }
        if constexpr (WP == 4) {
        // pieces ct, ct + 128, ...: the row advances by 32 per step, so the row's position inside its group of eight
        // (hence the swizzle) is the thread's own; the pieces of a batch are loaded before any is expanded
        const uint4* src = reinterpret_cast<const uint4*>(S.bp[stage]) + ct;
        const int n_lo = (ct >> 2) & 7, pp = ct & 3;
        uint8_t* row = S.b[bstage] + uint32_t(ct >> 5) * 1024u + uint32_t(n_lo) * 128u;
        uint8_t* d0 = row + (uint32_t((2 * pp) ^ n_lo) << 4);
        uint8_t* d1 = row + (uint32_t((2 * pp + 1) ^ n_lo) << 4);
        constexpr int kBatch = 2, kSteps = BN * 4 / kConvThreads;          // 32-row steps per thread
        static_assert(kSteps % kBatch == 0, "converter batches must divide the tile");
#pragma unroll 1
        for (int i0 = 0; i0 < kSteps; i0 += kBatch) {
          uint4 w[kBatch];
#pragma unroll
          for (int u = 0; u < kBatch; ++u) w[u] = src[(i0 + u) * kConvThreads];
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const uint32_t in[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
            uint32_t o[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint32_t lo = in[i] & 0x0F0F0F0Fu, hi = (in[i] >> 4) & 0x0F0F0F0Fu;
              o[2 * i] = __byte_perm(lo, hi, 0x5140);
              o[2 * i + 1] = __byte_perm(lo, hi, 0x7362);
            }
            *reinterpret_cast<uint4*>(d0 + (i0 + u) * 4096) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4*>(d1 + (i0 + u) * 4096) = make_uint4(o[4], o[5], o[6], o[7]);
          }
        }
        } else {
        // 6-bit codes: a packed row is 96 bytes; output piece p of row n (16 codes) comes from the 12 bytes at 12 p of
        // that row.  Thread ct takes pieces ct, ct + 128, ...: row (ct >> 3) + 16 per step, piece ct & 7.  The three
        // words of a warp's 32 pieces fall on 32 different banks (word index 24 n + 3 p).
        const int n_lo = (ct >> 3) & 7, pc = ct & 7;
        const uint32_t* src = reinterpret_cast<const uint32_t*>(S.bp[stage]) + (ct >> 3) * 24 + pc * 3;
        uint8_t* dst = S.b[bstage] + uint32_t(ct >> 6) * 1024u + uint32_t(n_lo) * 128u + (uint32_t(pc ^ n_lo) << 4);
        constexpr int kSteps = BN * 8 / kConvThreads;                      // 16-row steps per thread
        auto spread = [](uint32_t f) {      // four 6-bit fields of f[23:0] -> four bytes
          return (f & 0x3Fu) | ((f & 0xFC0u) << 2) | ((f & 0x3F000u) << 4) | ((f & 0xFC0000u) << 6);
        };
#pragma unroll 2
        for (int i = 0; i < kSteps; ++i) {
          const uint32_t w0 = src[i * 16 * 24], w1 = src[i * 16 * 24 + 1], w2 = src[i * 16 * 24 + 2];
          const uint32_t o0 = spread(w0), o1 = spread(__funnelshift_r(w0, w1, 24)), o2 = spread(__funnelshift_r(w1, w2, 16)),
                         o3 = spread(w2 >> 8);
          *reinterpret_cast<uint4*>(dst + i * 2048) = make_uint4(o0, o1, o2, o3);
        }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&S.ready[bstage]));
        if (++stage == kStages) { stage = 0; phase ^= 1; }
        if (++bstage == Storage::kStagesB) { bstage = 0; bphase ^= 1; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - 2;                     // 0..15
    const int quarter = warp & 3;                // TMEM lane quarter this warp may read
    const int slice = ew >> 2;                   // which 64 accumulator columns
    const bool slice_on = slice * kSliceCols < BN;
    const EpilogueParams& ep = P.ep;
    const int kza = P.K * ep.z_a;
    const bool res16 = ep.residual != nullptr && ep.residual_bf16;
    const bool res32 = ep.residual != nullptr && !ep.residual_bf16;
    // the common epilogue applies the pair step it was compiled with; any other combination goes chunk by chunk
    const bool fast_ok = ep.acc_debug == nullptr && (ep.rope != nullptr) == (PAIR == kPairRope) && (ep.glu != 0) == (PAIR == kPairGlu);
    const bool sat = ep.qmax <= 127;             // byte codes narrow enough for the comparison-free quantizer
    const bool direct = P.direct_requant != 0;
    const int cl0 = slice * kSliceCols;          // first column of this warp inside the tile
    ColTerms& C = S.cols[ew];
    // Raw per-column inputs of the warp's slice (lane: columns lane and lane + 32 of the slice) and the row's code
    // sum, fetched one tile ahead; nothing is computed from them before the next tile starts, so the loads stay in
    // flight behind this tile's epilogue.
    int nx_zw[2] = {0, 0}, nx_ws[2] = {0, 0}, nx_asum = 0;
    float nx_sw[2] = {0.f, 0.f}, nx_bs[2] = {0.f, 0.f};
    auto fetch_terms = [&](int t) {
      if (t >= tiles || !slice_on) return;
      const TileOrigin o = tile_origin(t, P.order, BN);
      const int tm0 = o.m0, tn0 = o.n0;
      // plain loads from clamped indices: nothing here may consume a loaded value (a select on it would hold the
      // warp until the load returns); rows and columns outside the matrix are dealt with where the values are used
      const int64_t tm = min(int64_t(tm0) + quarter * 32 + lane, int64_t(P.M) - 1);
      nx_asum = __ldg(P.asum + tm);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int j = min(tn0 + cl0 + lane + 32 * h, P.N - 1);
        if (ep.z_w) nx_zw[h] = __ldg(ep.z_w + j);
        nx_ws[h] = __ldg(P.wsum + j);
        if (ep.s_w) nx_sw[h] = __ldg(ep.s_w + j);
        if (ep.bias) nx_bs[h] = __ldg(ep.bias + j);
      }
    };
    // bulk copy of the residual box of tile t (rows and columns outside the matrix are zero-filled)
    const uint32_t res_buf = smem_u32(S.res) + uint32_t(RES ? ew : 0) * kResBytes;
    const uint32_t res_bar = smem_u32(&S.res_full[ew]);
    bool res_pending = false;
    auto fetch_residual = [&](int t) {
      if (!RES || t >= tiles || !slice_on) return;
      const TileOrigin o = tile_origin(t, P.order, BN);
      const int tm0 = o.m0, tn0 = o.n0;
      if (lane == 0) {
        // the box's last content may still be on its way out (the bulk store of the previous tile reads it)
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        mbar_expect_tx(res_bar, kResBytes);
        tma_load_2d(res_buf, &map_res, res_bar, tn0 + cl0, tm0 + quarter * 32);
      }
      res_pending = true;
    };
    fetch_residual(blockIdx.x);
    fetch_terms(blockIdx.x);
    int it = 0;
    for (int tile = blockIdx.x; tile < tiles && !*abort; tile += gridDim.x, ++it) {
      const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
      const TileOrigin o = tile_origin(tile, P.order, BN);
      const int m0 = o.m0, n0 = o.n0;
      const int64_t m = int64_t(m0) + quarter * 32 + lane;
      const bool row_ok = m < P.M;
      // warp-uniform: whole 64-column slice inside the matrix, common epilogue (rows beyond M are clipped by
      // the bulk store)
      const bool any_row = m0 + quarter * 32 < P.M;          // warp-uniform: at least one valid row
      const bool fast = fast_ok && slice_on && n0 + cl0 + kSliceCols <= P.N && any_row;
      // bf16 residual of the slice: requested now, needed only after the main loop of the tile
      // (the pieces of two chunks at a time, in one set of registers: those of the first two chunks are requested here,
      // those of the next two as soon as the first two have been added, a chunk's store and the next chunk's accumulator
      // load ahead of their use; every index into the register array is a compile-time one)
      constexpr int kPairPieces = 2 * (kChunk / 8);
      uint4 res[kPairPieces];
      // (float outputs: that is where a residual stream is added; a code output with a residual loads the pieces where
      // they are used)
      constexpr bool kResRegs = !RES && (OUT == kOutF32 || OUT == kOutBf16);
      const bool res_regs = kResRegs && fast && res16 && row_ok;
      const uint4* res_ptr = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(ep.residual) + m * ep.ld_residual + n0 + cl0);
      if (res_regs) {
#pragma unroll
        for (int i = 0; i < kPairPieces; ++i) res[i] = __ldg(res_ptr + i);
      }
      // corr = acc - z_w (asum - K z_a) - z_a wsum; this tile's inputs were fetched during the previous tile
      const int32_t asum_c = row_ok ? nx_asum - kza : 0;
      // stage the per-column terms of the warp's slice in the warp's own buffer (read by this warp alone)
      if (slice_on) {
        __syncwarp();                                          // the previous tile's reads of the buffer are done
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int cs = lane + 32 * h, j = n0 + cl0 + cs;
          const bool in = j < P.N;                             // columns outside the matrix: all terms 0
          float sc = in ? ep.scale_a * (ep.s_w ? nx_sw[h] : ep.s_w_scalar) : 0.f, bi = in && ep.bias ? nx_bs[h] : 0.f;
          if (direct) {
            const int gw = ep.group_width;
            const int gi = (j >= gw) + (j >= 2 * gw) + (j >= 3 * gw);
            const float inv = gi == 0 ? ep.inv_out_scale[0] : gi == 1 ? ep.inv_out_scale[1] : gi == 2 ? ep.inv_out_scale[2] : ep.inv_out_scale[3];
            sc *= inv;
            bi *= inv;
          }
          C.nzw[cs] = in ? -(ep.z_w ? nx_zw[h] : ep.z_w_scalar) : 0;
          C.kw[cs] = in ? -ep.z_a * nx_ws[h] : 0;
          C.sc[cs] = sc;
          C.bi[cs] = bi;
        }
        __syncwarp();
      }
      fetch_terms(tile + int(gridDim.x));                    // next tile's inputs: in flight during this epilogue
      int code_sum = 0;
      // rotary embedding: this row's line of the (cos, sin) table and the slice's first column inside its head
      const float2* rope_row = nullptr;
      int rope_hb = 0;
      if (PAIR == kPairRope && n0 + cl0 < ep.rope_cols) {
        rope_row = ep.rope + int64_t(m % ep.rope_period) * (ep.rope_dim >> 1);
        rope_hb = (n0 + cl0) % ep.rope_dim;
      }

      if (!mbar_wait(smem_u32(&S.tmem_full[acc]), acc_phase, abort, 4)) break;
      tc_fence_after();
      const uint32_t taddr0 = tmem_base + (uint32_t(quarter * 32) << 16) + acc * kAccStride + cl0;
      if (RES && res_pending) {
        if (!mbar_wait(res_bar, uint32_t(it) & 1u, abort, 6)) break;
        res_pending = false;
      }
      if (fast) {
        // (two chunks per trip: unrolled further, the 16 values of four chunks in flight spill at 96 registers)
        static_assert(kSliceChunks % 2 == 0, "the chunk loop takes two chunks per trip");
#pragma unroll 1
        for (int cp = 0; cp < kSliceChunks; cp += 2) {
#pragma unroll
        for (int cu = 0; cu < 2; ++cu) {
          const int c = cp + cu;
          const int cl = cl0 + c * kChunk;                     // column inside the tile
          const int col0 = n0 + cl;
          uint32_t r[kChunk];
          tmem_ld16(taddr0 + c * kChunk, r);
          tmem_ld_wait();
          float v[kChunk];
#pragma unroll
          for (int q4 = 0; q4 < kChunk / 4; ++q4) {
            const int4 nz = *reinterpret_cast<const int4*>(&C.nzw[c * kChunk + 4 * q4]);
            const int4 kw = *reinterpret_cast<const int4*>(&C.kw[c * kChunk + 4 * q4]);
            const float4 sc = *reinterpret_cast<const float4*>(&C.sc[c * kChunk + 4 * q4]);
            const float4 bi = *reinterpret_cast<const float4*>(&C.bi[c * kChunk + 4 * q4]);
            const float f0 = float(int32_t(r[4 * q4 + 0]) + nz.x * asum_c + kw.x), f1 = float(int32_t(r[4 * q4 + 1]) + nz.y * asum_c + kw.y);
            const float f2 = float(int32_t(r[4 * q4 + 2]) + nz.z * asum_c + kw.z), f3 = float(int32_t(r[4 * q4 + 3]) + nz.w * asum_c + kw.w);
            unpack2(fma2(pack2(sc.x, sc.y), pack2(f0, f1), pack2(bi.x, bi.y)), v[4 * q4 + 0], v[4 * q4 + 1]);
            unpack2(fma2(pack2(sc.z, sc.w), pack2(f2, f3), pack2(bi.z, bi.w)), v[4 * q4 + 2], v[4 * q4 + 3]);
          }
          if (ep.gelu) {
#pragma unroll
            for (int e = 0; e < kChunk; e += 2) gelu_erf_pair(v[e], v[e + 1]);
          }
          if (res32 && row_ok) {
            // float32 residual: read where it is used (16 columns = four 16-byte loads of this thread's row)
            const float4* rp = reinterpret_cast<const float4*>(static_cast<const float*>(ep.residual) + m * ep.ld_residual + col0);
#pragma unroll
            for (int i = 0; i < kChunk / 4; ++i) {
              const float4 r4 = __ldg(rp + i);
              v[4 * i] += r4.x; v[4 * i + 1] += r4.y; v[4 * i + 2] += r4.z; v[4 * i + 3] += r4.w;
            }
          }
          if (res16 && row_ok) {
#pragma unroll
            for (int i = 0; i < kChunk / 8; ++i) {
              uint4 w4;
              if (RES) {
                // the thread's row of the box: 16-byte piece p sits at (p ^ (row & 7)) inside the 128-byte row
                const uint32_t piece = uint32_t(c * (kChunk / 8) + i);
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w4.x), "=r"(w4.y), "=r"(w4.z), "=r"(w4.w)
                             : "r"(res_buf + uint32_t(lane) * 128u + ((piece ^ uint32_t(lane & 7)) << 4)));
              } else {
                w4 = kResRegs ? res[cu * (kChunk / 8) + i] : __ldg(res_ptr + c * (kChunk / 8) + i);
              }
              const uint32_t ws[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
              for (int k = 0; k < 4; ++k)
                unpack2(add2(pack2(v[i * 8 + 2 * k], v[i * 8 + 2 * k + 1]), pack2(__uint_as_float(ws[k] << 16), __uint_as_float(ws[k] & 0xffff0000u))),
                        v[i * 8 + 2 * k], v[i * 8 + 2 * k + 1]);
            }
          }
          if (cu == 1 && res_regs && cp + 2 < kSliceChunks) {      // both chunks of the pair have taken their pieces
#pragma unroll
            for (int i = 0; i < kPairPieces; ++i) res[i] = __ldg(res_ptr + (cp + 2) * (kChunk / 8) + i);
          }
          if (PAIR == kPairRope && rope_row != nullptr && col0 < ep.rope_cols) {       // warp-uniform: range edges fall on chunk edges
            int hx = rope_hb + c * kChunk;
            while (hx >= ep.rope_dim) hx -= ep.rope_dim;
            const float4* cs = reinterpret_cast<const float4*>(rope_row + (hx >> 1));
#pragma unroll
            for (int i = 0; i < kChunk / 4; ++i) {
              const float4 t4 = __ldg(cs + i);
              rope_rotate(make_float2(t4.x, t4.y), v[4 * i], v[4 * i + 1]);
              rope_rotate(make_float2(t4.z, t4.w), v[4 * i + 2], v[4 * i + 3]);
            }
          }
          ChunkQuant q{};
          if constexpr (OUT == kOutC4 || OUT == kOutC8) q = chunk_quant(ep, P, col0);
          if constexpr (OUT == kOutC8 && PAIR == kPairGlu) {
            {
              // gated product: 16 accumulator columns (gate, up interleaved) give 8 byte codes; the slice's 32 codes
              // fill one box row
              const float magic = __uint_as_float(kMagicBits);
              uint32_t u[kChunk / 2];
#pragma unroll
              for (int i = 0; i < kChunk / 2; ++i) {
                const float t = fminf(fmaxf(silu_mul(v[2 * i], v[2 * i + 1]) * q.mult, q.lo), q.hi);
                u[i] = __float_as_uint(t + magic);
              }
              uint32_t w[2];
#pragma unroll
              for (int i = 0; i < 2; ++i) {
                w[i] = __vadd4(__byte_perm(__byte_perm(u[4 * i], u[4 * i + 1], 0x0040), __byte_perm(u[4 * i + 2], u[4 * i + 3], 0x0040), 0x5410), q.z4);
                code_sum += __dp4a(w[i], 0x01010101u, 0u);
              }
              const uint32_t buf = smem_u32(S.epi[ew]);
              if (c == 0) box_begin(lane);
              sts64(box_slot(buf, lane, c >> 1) + uint32_t(c & 1) * 8u, w[0], w[1]);
              if (c == kSliceChunks - 1) box_end(&map_out, buf, lane, (col0 - (kSliceChunks - 1) * kChunk) >> 1, m0 + quarter * 32);
              continue;
            }
          }
          if constexpr (RES && OUT == kOutBf16) {
            // in place: the 16 output values take the two 16-byte pieces their residual values came from
            uint32_t w[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
              w[k] = *reinterpret_cast<const uint32_t*>(&h);
            }
#pragma unroll
            for (int i = 0; i < kChunk / 8; ++i) {
              const uint32_t piece = uint32_t(c * (kChunk / 8) + i);
              sts128(res_buf + uint32_t(lane) * 128u + ((piece ^ uint32_t(lane & 7)) << 4), w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
            }
            if (c == kSliceChunks - 1) {
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (lane == 0) {
                tma_store_2d(&map_out, res_buf, n0 + cl0, m0 + quarter * 32);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
              }
            }
            continue;
          }
          if constexpr (!(RES && OUT == kOutBf16))
            emit_chunk<OUT>(&map_out, smem_u32(S.epi[ew]), lane, q, v, c, col0, m0 + quarter * 32, code_sum, direct, sat);
        }
        }
      } else if (slice_on && any_row && n0 + cl0 < P.N) {
#pragma unroll 1
        for (int c = 0; c < kSliceChunks; ++c) {
          const int cl = cl0 + c * kChunk;
          uint32_t r[kChunk];
          __syncwarp();
          tmem_ld16(taddr0 + c * kChunk, r);
          tmem_ld_wait();
          if (row_ok && n0 + cl < P.N) slow_chunk(ep, P, C, r, c * kChunk, m, n0 + cl, asum_c, &code_sum);
        }
      }
      // accumulator buffer free again
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.tmem_empty[acc]));
      fetch_residual(tile + int(gridDim.x));               // every lane has read this tile's box (the __syncwarp above)
      if (ep.out_row_sum != nullptr && row_ok && code_sum != 0) atomicAdd(ep.out_row_sum + m, code_sum);
    }
    if (RES && res_pending) mbar_drain(res_bar, uint32_t(it) & 1u);              // left the loop early: the copy must land
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");     // bulk stores complete
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

// Operand tensor map: rows of `row_bytes` bytes, boxes of `box_bytes` x box_rows; byte tiles take the 128-byte swizzle
// of the MMA descriptor, packed tiles (expanded by the converter warps) stay unswizzled.
repq_status make_map(CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t row_bytes, int64_t ld, int box_rows,
                     int box_bytes = BK, bool swizzle = true) {
  EncodeTiledFn fn = encode_fn();
  REPQ_REQUIRE(fn != nullptr, REPQ_CUDA_ERROR, "qgemm: cuTensorMapEncodeTiled is not available");
  const cuuint64_t dims[2] = {cuuint64_t(row_bytes), cuuint64_t(rows)};
  const cuuint64_t strides[1] = {cuuint64_t(ld)};
  const cuuint32_t box[2] = {cuuint32_t(box_bytes), cuuint32_t(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
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
  L.off_a = packed4(d.bits_a) ? bump(size_t(d.M) * L.ld_a) : 0;
  L.off_w = 0;                                  // packed weights are expanded inside the kernel
  L.off_asum = d.a_row_sum ? 0 : bump(size_t(d.M) * 4);
  L.off_wsum = d.w_row_sum ? 0 : bump(size_t(d.N) * 4);
  L.total = cur;
  return L;
}

// Tile width: rounds of tiles over the SMs times the time of one round, which has a part that does not depend on the
// width (per-tile waits, staging and bulk-store latencies of the epilogue warps) and a part proportional to it
// (measured: about 160 columns' worth of fixed time for K = 768).
// Whether a launch takes its bf16 residual through bulk-copied boxes (tiles of at most 192 columns, short K).
bool residual_boxes(const TcParams& P) {
  const EpilogueParams& ep = P.ep;
  // (up to K = 3072: beyond, the main loop sets the pace, and its time per k-block does not shrink with the tile width
  // (the operand copies in flight, four stages, against the L2 latency), so that 256-column tiles win: measured at
  // 8192 x 4096 x 4096 101 us with 256 columns against 111 with 192, at 18464 x 1024 x 4096 67 against 79)
  return ep.out_kind == REPQ_OUT_BF16 && ep.residual != nullptr && ep.residual_bf16 && ep.acc_debug == nullptr &&
         ep.glu == 0 && P.K <= 3072 && !P.w_packed4;
}

int pick_bn(int M, int N, int K, int sms, bool w_packed4, bool res_boxes) {
  const int m_tiles = (M + BM - 1) / BM;
  int best = 256;
  long best_cost = -1;
  for (int bn : {256, 192, 128}) {
    if (w_packed4 && bn > kMaxBNW4) continue;
    const long tiles = long(m_tiles) * ((N + bn - 1) / bn);
    const long rounds = (tiles + sms - 1) / sms;
    // a round costs its width plus a fixed part; where the epilogue adds a bf16 residual at short K, a round is the longer
    // of the main loop (0.34 us per k-block) and the epilogue, and the epilogue of a 256-column tile (residual by
    // row-per-lane loads) takes 1.7 x the time of a narrower one whose residual box was copied in a tile ahead (measured
    // at 18464 x 1024 x 1024: 39.6 us with 256 columns, 33.9 with 192)
    const long main_loop = 34L * ((K + BK - 1) / BK), epilogue = bn == 256 ? 950 : 550;
    const long cost = res_boxes ? rounds * (main_loop > epilogue ? main_loop : epilogue) : rounds * (bn + 160);
    if (best_cost < 0 || cost < best_cost) { best = bn; best_cost = cost; }
  }
  return best;
}

// Tensor map of the output for the epilogue's bulk stores: boxes of 32 rows x 32 bytes, 32-byte swizzle.
repq_status make_out_map(CUtensorMap* map, const TcParams& P) {
  EncodeTiledFn fn = encode_fn();
  REPQ_REQUIRE(fn != nullptr, REPQ_CUDA_ERROR, "qgemm: cuTensorMapEncodeTiled is not available");
  const EpilogueParams& ep = P.ep;
  CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_UINT8;
  cuuint64_t inner = cuuint64_t(ep.glu ? P.N / 2 : P.N), esz = 1;     // output columns
  if (ep.out_kind == REPQ_OUT_F32) { dt = CU_TENSOR_MAP_DATA_TYPE_FLOAT32; esz = 4; }
  else if (ep.out_kind == REPQ_OUT_BF16) { dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16; esz = 2; }
  else if (ep.pack4) inner /= 2;
  const cuuint64_t dims[2] = {inner, cuuint64_t(P.M)};
  const cuuint64_t strides[1] = {cuuint64_t(ep.ldo) * esz};
  const cuuint32_t box[2] = {cuuint32_t(32 / esz), 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, dt, 2, ep.out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  REPQ_REQUIRE(r == CUDA_SUCCESS, REPQ_CUDA_ERROR, "qgemm: output tensor map failed with code %d", int(r));
  return REPQ_OK;
}

// Tensor map of a bf16 matrix (the residual, the output) for the epilogue warps' boxes: 32 rows x 64 columns, 128-byte
// swizzle.
repq_status make_box_map(CUtensorMap* map, const TcParams& P, const void* base, int64_t ld) {
  EncodeTiledFn fn = encode_fn();
  REPQ_REQUIRE(fn != nullptr, REPQ_CUDA_ERROR, "qgemm: cuTensorMapEncodeTiled is not available");
  const cuuint64_t dims[2] = {cuuint64_t(P.N), cuuint64_t(P.M)};
  const cuuint64_t strides[1] = {cuuint64_t(ld) * 2};
  const cuuint32_t box[2] = {kSliceCols, 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  REPQ_REQUIRE(r == CUDA_SUCCESS, REPQ_CUDA_ERROR, "qgemm: box tensor map failed with code %d", int(r));
  return REPQ_OK;
}

template <int BN, int OUT, bool RES, int PAIR, int WP>
repq_status launch_tc_w(const CUtensorMap& map_a, const CUtensorMap& map_b, const TcParams& P, int sms, cudaStream_t st) {
  CUtensorMap map_out, map_res;
  if (RES) {
    REPQ_TRY(make_box_map(&map_res, P, P.ep.residual, P.ep.ld_residual));
    REPQ_TRY(make_box_map(&map_out, P, P.ep.out, P.ep.ldo));
  } else {
    REPQ_TRY(make_out_map(&map_out, P));
    map_res = map_out;                                     // not read
  }
  const size_t smem = sizeof(SharedStorage<BN, RES, WP>);
  REPQ_CUDA(cudaFuncSetAttribute(qgemm_tc_kernel<BN, OUT, RES, PAIR, WP>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  const int tiles = ((P.M + BM - 1) / BM) * ((P.N + BN - 1) / BN);
  const int grid = tiles < sms ? tiles : sms;
  REPQ_CUDA(launch_chained(qgemm_tc_kernel<BN, OUT, RES, PAIR, WP>, dim3(grid), dim3(kThreads), smem, st, map_a, map_b, map_out, map_res, P));
  note_launch();
  return REPQ_OK;
}

template <int BN, int OUT, bool RES, int PAIR = kPairNone>
repq_status launch_tc_res(const CUtensorMap& map_a, const CUtensorMap& map_b, const TcParams& P, int sms, cudaStream_t st) {
  if constexpr (!RES && BN <= kMaxBNW4) {
    if (P.w_packed4 == 4) return launch_tc_w<BN, OUT, false, PAIR, 4>(map_a, map_b, P, sms, st);
    if (P.w_packed4 == 6) return launch_tc_w<BN, OUT, false, PAIR, 6>(map_a, map_b, P, sms, st);
  }
  return launch_tc_w<BN, OUT, RES, PAIR, 0>(map_a, map_b, P, sms, st);
}

template <int BN, int OUT>
repq_status launch_tc_out(const CUtensorMap& map_a, const CUtensorMap& map_b, const TcParams& P, int sms, cudaStream_t st) {
  // bf16 outputs with a bf16 residual on tiles of at most 192 columns: the residual boxes, which also carry the output,
  // fit beside the four stages
  if constexpr (BN <= 192 && OUT == kOutBf16) {
    if (residual_boxes(P))
      return launch_tc_res<BN, OUT, true>(map_a, map_b, P, sms, st);
  }
  return launch_tc_res<BN, OUT, false>(map_a, map_b, P, sms, st);
}

template <int BN>
repq_status launch_tc(const CUtensorMap& map_a, const CUtensorMap& map_b, const TcParams& P, int sms, cudaStream_t st) {
  if (P.ep.out_kind == REPQ_OUT_F32) return launch_tc_out<BN, kOutF32>(map_a, map_b, P, sms, st);
  if (P.ep.out_kind == REPQ_OUT_BF16) return launch_tc_out<BN, kOutBf16>(map_a, map_b, P, sms, st);
  if (P.ep.pack4) return launch_tc_out<BN, kOutC4>(map_a, map_b, P, sms, st);
  if (P.ep.rope != nullptr) return launch_tc_res<BN, kOutC8, false, kPairRope>(map_a, map_b, P, sms, st);
  if (P.ep.glu) return launch_tc_res<BN, kOutC8, false, kPairGlu>(map_a, map_b, P, sms, st);
  return launch_tc_out<BN, kOutC8>(map_a, map_b, P, sms, st);
}

// A wait that nothing ends: one thread sets up an mbarrier that never receives its arrival and waits on it through the
// same bounded-wait routine as the tensor-core kernels, with the caller's limit.  The wait runs out, the status word
// takes the code, the kernel returns.
__global__ void wait_selftest_kernel(long long limit_cycles, int code) {
  __shared__ alignas(8) uint64_t bar;
  __shared__ volatile int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc::mbar_wait(smem_u32(&bar), 0, &abort_flag, code, &g_status_word, limit_cycles);
  }
}

}  // namespace

repq_status launch_wait_selftest(long long limit_cycles, cudaStream_t st) {
  REPQ_REQUIRE(device_status_word() != nullptr, REPQ_CUDA_ERROR, "wait_selftest: device status word unavailable");
  wait_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles, 77);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

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
  if (!packed4(d.bits_a) && !(aligned(d.a_codes, 16) && d.lda_bytes % 16 == 0)) return false;
  if (!(aligned(d.w_codes, 16) && d.ldw_bytes % 16 == 0)) return false;      // byte or packed: the tiles come by TMA
  const int64_t obytes = d.out_kind == REPQ_OUT_F32 ? 4 : d.out_kind == REPQ_OUT_BF16 ? 2 : 1;
  if (!aligned(d.out, 16) || (d.ldo * obytes) % 16 != 0) return false;
  if (d.out_kind == REPQ_OUT_CODES && (d.N / d.out_groups) % kChunk != 0) return false;   // one quantizer per 16-column chunk
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
  if (packed4(d.bits_a)) {
    REPQ_TRY(launch_expand4(d.a_codes, d.M, d.K, d.lda_bytes, w8 + L.off_a, L.ld_a, L.ld_a, st));
    a = w8 + L.off_a; lda = L.ld_a;
  }
  TcParams P{};
  P.w_packed4 = packed4(d.bits_w) ? 4 : packed6(d.bits_w) ? 6 : 0;
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
  P.direct_requant = d.out_kind == REPQ_OUT_CODES && !d.gelu && !d.residual && !d.glu;
  REPQ_REQUIRE(device_status_word() != nullptr, REPQ_CUDA_ERROR, "qgemm: device status word unavailable");
  const int sms = sm_count();
  const int bn = pick_bn(d.M, d.N, d.K, sms, P.w_packed4 != 0, residual_boxes(P));
  {
    // panels of activations: all row tiles while the activations take at most 40 MB (a third of the L2 capacity),
    // else about 24 MB (measured at 8192 x 4096 x 11008 with residual: 248 us with 40 MB panels, 240-242 with
    // 12..30 MB: the weight tiles and the residual / output rows stream through the same L2), at least 8 row tiles
    const int m_tiles = (d.M + BM - 1) / BM, n_tiles = (d.N + bn - 1) / bn;
    const int64_t a_bytes = int64_t(d.M) * d.K;
    const int64_t fit = (int64_t(a_bytes <= (int64_t(40) << 20) ? 40 : 24) << 20) / (int64_t(BM) * d.K);
    int panel = int(fit < 8 ? 8 : fit);
    if (panel > m_tiles) panel = m_tiles;
    TileOrder& T = P.order;
    T.panel = panel;
    T.m_tiles = m_tiles;
    T.last_rows = m_tiles - (m_tiles / panel) * panel;
    T.full = (m_tiles / panel) * panel * n_tiles;
    const uint64_t tiles = uint64_t(m_tiles) * uint64_t(n_tiles);
    T.by_panel_tiles = fast_div(uint32_t(panel) * uint32_t(n_tiles), tiles);
    T.by_panel = fast_div(uint32_t(panel), tiles);
    T.by_last_rows = fast_div(uint32_t(T.last_rows > 0 ? T.last_rows : 1), tiles);
  }
  CUtensorMap map_a, map_b;
  REPQ_TRY(make_map(&map_a, a, d.M, d.K, lda, BM));
  if (P.w_packed4) REPQ_TRY(make_map(&map_b, d.w_codes, d.N, code_row_bytes(d.K, d.bits_w), d.ldw_bytes, bn, BK * P.w_packed4 / 8, false));
  else REPQ_TRY(make_map(&map_b, d.w_codes, d.N, d.K, d.ldw_bytes, bn));
  if (bn == 256) return launch_tc<256>(map_a, map_b, P, sms, st);
  if (bn == 192) return launch_tc<192>(map_a, map_b, P, sms, st);
  return launch_tc<128>(map_a, map_b, P, sms, st);
}

}  // namespace repq
