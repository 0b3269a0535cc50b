// P.V with log2-domain Softmax codes (Eqs. 16-17): A^ = s 2^(-ceil(p/2)) (sqrt2 if p odd else 1).
//
// Codes are turned into exact bf16 powers of two and fed to warp-level bf16 MMA with fp32 accumulation.
// Even and odd codes go to two separate accumulators, so both MMA operands are exact (powers of two; small
// integers v - z_v) and the irrational factor sqrt2 of Eq. 17 is applied once, in float32, to the odd
// accumulator:  O = s s_v (acc_even + sqrt2 acc_odd).
//
// The code -> operand map is a 256-entry table in shared memory built once per CTA: for 4-bit codes it is
// indexed by a whole byte (two codes) and returns the packed bf16 pair for the even and for the odd
// accumulator; for 6/8-bit codes it is indexed by one code.  A CTA of 8 warps owns 128 query rows (64 when
// the head is wider than 64) of one (batch, head) pair.  V is staged in shared memory as bf16 (v - z_v), up
// to 256 keys at a time; the codes of the next 64 keys are fetched into registers while the current 64 are
// multiplied.  Key order inside a 64-key chunk is permuted so that every thread owns 16 consecutive codes of
// its two query rows (one 64-bit or 128-bit load); the V fragments are fetched with ldmatrix.trans using the
// same permutation of row addresses.  Keys beyond Lk need no masking (their V rows are zero); under a
// causal mask only the chunks that touch the diagonal are masked element by element.
#include <cuda_bf16.h>

#include "kernels.h"

namespace repq {
namespace {

constexpr int kKeys = 64;       // keys per MMA chunk
constexpr int kVKeys = 256;     // keys of V resident in shared memory
constexpr int kThreads = 256;

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
  const uint32_t addr = uint32_t(__cvta_generic_to_shared(smem_row));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// bf16 bit pattern of 2^(-ceil(c/2)); zero once the exponent leaves the normal range.
__device__ __forceinline__ uint32_t pow2_bits(uint32_t c) {
  const uint32_t e = (c + 1u) >> 1;
  return e <= 126u ? (127u - e) << 7 : 0u;
}

// Operands of two consecutive codes: .x = bf16 pair for the even accumulator, .y = for the odd one.
template <bool kP4>
__device__ __forceinline__ uint2 lookup_pair(const uint2* lut4, const uint32_t* lut8, uint32_t codes) {
  if (kP4) return lut4[codes & 0xFFu];
  const uint32_t l0 = lut8[codes & 0xFFu], l1 = lut8[(codes >> 8) & 0xFFu];
  return make_uint2(__byte_perm(l0, l1, 0x5410), __byte_perm(l0, l1, 0x7632));
}

// NG = number of 64-wide column groups of V handled by the CTA (d_h <= 64 * NG); 8 / NG warps per group.
template <int NG, bool kP4>
__global__ void __launch_bounds__(kThreads)
pv_kernel(PvParams P) {
  constexpr int kDhp = 64 * NG;
  constexpr int kVStride = kDhp + 8;                     // bf16 elements; conflict-free ldmatrix rows
  constexpr int kRowWarps = 8 / NG;
  constexpr int kQRows = 16 * kRowWarps;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __nv_bfloat16* sV = reinterpret_cast<__nv_bfloat16*>(smem_raw);     // [kVKeys][kVStride]
  __shared__ uint2 lut4[256];
  uint32_t* lut8 = reinterpret_cast<uint32_t*>(lut4);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  {
    const uint32_t i = uint32_t(tid);
    if (kP4) {
      const uint32_t c0 = i & 15u, c1 = i >> 4, b0 = pow2_bits(c0), b1 = pow2_bits(c1);
      lut4[i] = make_uint2(((c0 & 1u) ? 0u : b0) | (((c1 & 1u) ? 0u : b1) << 16),
                           ((c0 & 1u) ? b0 : 0u) | (((c1 & 1u) ? b1 : 0u) << 16));
    } else {
      const uint32_t b = pow2_bits(i);
      lut8[i] = (i & 1u) ? (b << 16) : b;
    }
  }
  const int rw = warp % kRowWarps;                        // row group of the warp
  const int cg = warp / kRowWarps;                        // column group of the warp
  const int g = lane >> 2, t = lane & 3;
  const int pair = blockIdx.y;
  const int bo = pair / P.batch_inner, bi = pair % P.batch_inner;
  const int q0 = blockIdx.x * kQRows;
  const uint8_t* p_base = P.p + int64_t(pair) * P.p_pair;
  const uint8_t* v_base = P.v + bo * P.v_so + bi * P.v_si;

  const int row_a = q0 + rw * 16 + g, row_b = row_a + 8;
  const int shift = P.Lk - P.Lq;
  // keys a row may attend to; rows beyond Lq produce values that are never stored
  const int valid_a = P.causal ? max(0, min(P.Lk, row_a + 1 + shift)) : P.Lk;
  const int valid_b = P.causal ? max(0, min(P.Lk, row_b + 1 + shift)) : P.Lk;
  const int warp_min_valid = P.causal ? max(0, min(P.Lk, q0 + rw * 16 + 1 + shift)) : P.Lk;
  int k_end = P.Lk;
  if (P.causal) k_end = max(0, min(P.Lk, min(q0 + kQRows, P.Lq) + shift));

  float acc_e[8][4], acc_o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc_e[j][e] = acc_o[j][e] = 0.f;

  constexpr int kCodeBytes = kP4 ? 8 : 16;               // bytes holding a thread's 16 codes
  const uint8_t* pa = p_base + int64_t(row_a < P.Lq ? row_a : 0) * P.ldp + t * kCodeBytes;
  const uint8_t* pb = p_base + int64_t(row_b < P.Lq ? row_b : 0) * P.ldp + t * kCodeBytes;

  // this thread's 16 codes of each of its two rows for the chunk starting at key k0 (keys k0 + 16 t .. + 15)
  auto load_codes = [&](int k0, uint32_t (&ca)[4], uint32_t (&cb)[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) ca[i] = cb[i] = 0u;
    if (k0 >= k_end) return;
    const int64_t boff = kP4 ? k0 / 2 : k0;               // bytes from the row start to chunk k0
    if (boff + t * kCodeBytes + kCodeBytes <= P.ldp) {
      if (kP4) {
        const uint2 wa = __ldcs(reinterpret_cast<const uint2*>(pa + boff)); ca[0] = wa.x; ca[1] = wa.y;
        const uint2 wb = __ldcs(reinterpret_cast<const uint2*>(pb + boff)); cb[0] = wb.x; cb[1] = wb.y;
      } else {
        const uint4 wa = __ldcs(reinterpret_cast<const uint4*>(pa + boff)); ca[0] = wa.x; ca[1] = wa.y; ca[2] = wa.z; ca[3] = wa.w;
        const uint4 wb = __ldcs(reinterpret_cast<const uint4*>(pb + boff)); cb[0] = wb.x; cb[1] = wb.y; cb[2] = wb.z; cb[3] = wb.w;
      }
    } else {
      // ragged end of the row: byte loads inside the row stride
      for (int e = 0; e < kCodeBytes; ++e) {
        if (boff + t * kCodeBytes + e < P.ldp) {
          ca[e >> 2] |= uint32_t(pa[boff + e]) << (8 * (e & 3));
          cb[e >> 2] |= uint32_t(pb[boff + e]) << (8 * (e & 3));
        }
      }
    }
  };

  uint32_t ca[4], cb[4];
  load_codes(0, ca, cb);

  for (int kv0 = 0; kv0 < k_end; kv0 += kVKeys) {
    // ---- up to 256 keys of V -> shared memory as bf16 (v - z_v); zero rows beyond Lk, zero columns beyond d_h
    __syncthreads();
    {
      constexpr int kGroupsPerRow = kDhp / 8;              // 8 columns per work item
      constexpr int kItems = kVKeys * kGroupsPerRow / kThreads;
      const int keys_here = min(kVKeys, (k_end - kv0 + kKeys - 1) / kKeys * kKeys);
      const int n_items = keys_here * kGroupsPerRow;
      // all loads of the thread are issued before the first conversion
      uint2 raw[kItems];
#pragma unroll
      for (int i = 0; i < kItems; ++i) {
        const int w = tid + i * kThreads;
        const int kr = w / kGroupsPerRow, c0 = (w % kGroupsPerRow) * 8;
        const int key = kv0 + kr;
        raw[i] = make_uint2(0u, 0u);
        if (w < n_items && key < P.Lk && c0 < P.d_h) {
          const uint8_t* vr = v_base + int64_t(key) * P.ldv;
          if (P.bits_v == 4) {
            const uint8_t* s = vr + c0 / 2;
            if ((reinterpret_cast<uintptr_t>(s) & 3) == 0 && c0 + 8 <= P.d_h) raw[i].x = __ldg(reinterpret_cast<const uint32_t*>(s));
            else for (int e = 0; e < 4; ++e) if (c0 + 2 * e < P.d_h) raw[i].x |= uint32_t(s[e]) << (8 * e);
          } else {
            const uint8_t* s = vr + c0;
            if ((reinterpret_cast<uintptr_t>(s) & 7) == 0 && c0 + 8 <= P.d_h) raw[i] = __ldg(reinterpret_cast<const uint2*>(s));
            else for (int e = 0; e < 8; ++e) if (c0 + e < P.d_h) (e < 4 ? raw[i].x : raw[i].y) |= uint32_t(s[e]) << (8 * (e & 3));
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kItems; ++i) {
        const int w = tid + i * kThreads;
        if (w >= n_items) continue;
        const int kr = w / kGroupsPerRow, c0 = (w % kGroupsPerRow) * 8;
        const int key = kv0 + kr;
        uint32_t o[4] = {0, 0, 0, 0};
        if (key < P.Lk && c0 < P.d_h) {
          int q[8];
          if (P.bits_v == 4) {
#pragma unroll
            for (int e = 0; e < 8; ++e) q[e] = int((raw[i].x >> (4 * e)) & 15u);
          } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) { q[e] = int((raw[i].x >> (8 * e)) & 255u); q[4 + e] = int((raw[i].y >> (8 * e)) & 255u); }
          }
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            const float f0 = c0 + e < P.d_h ? float(q[e] - P.z_v) : 0.f;
            const float f1 = c0 + e + 1 < P.d_h ? float(q[e + 1] - P.z_v) : 0.f;
            const __nv_bfloat162 h = __floats2bfloat162_rn(f0, f1);
            o[e >> 1] = *reinterpret_cast<const uint32_t*>(&h);
          }
        }
        *reinterpret_cast<uint4*>(&sV[kr * kVStride + c0]) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
    __syncthreads();

    const int kv_end = min(k_end, kv0 + kVKeys);
    for (int k0 = kv0; k0 < kv_end; k0 += kKeys) {
      uint32_t na[4], nb[4];
      load_codes(k0 + kKeys, na, nb);                       // next chunk's codes, in flight during the MMAs
      const bool need_mask = k0 + kKeys > warp_min_valid;   // warp-uniform: this chunk touches the causal diagonal
      // ---- 4 MMA k-steps of 16 keys; step s uses codes 4s..4s+3 of every thread
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        if (k0 + 4 * s >= k_end) break;                     // every key of this step (k0 + 16 t + 4 s + i) is past the end
        // the 4 codes of this step, per row: 16 bits (4-bit codes) or 32 bits (byte codes)
        uint32_t qa, qb;
        if (kP4) {
          qa = (ca[s >> 1] >> (16 * (s & 1))) & 0xffffu;
          qb = (cb[s >> 1] >> (16 * (s & 1))) & 0xffffu;
        } else {
          qa = ca[s];
          qb = cb[s];
        }
        constexpr int kPairShift = kP4 ? 8 : 16;            // bits per pair of codes
        // fragment order: a0 = (row g, k 2t..), a1 = (row g+8, k 2t..), a2 = (row g, k 2t+8..), a3 = (row g+8, k 2t+8..)
        const uint2 fa0 = lookup_pair<kP4>(lut4, lut8, qa), fa1 = lookup_pair<kP4>(lut4, lut8, qa >> kPairShift);
        const uint2 fb0 = lookup_pair<kP4>(lut4, lut8, qb), fb1 = lookup_pair<kP4>(lut4, lut8, qb >> kPairShift);
        uint32_t ae[4] = {fa0.x, fb0.x, fa1.x, fb1.x};
        uint32_t ao[4] = {fa0.y, fb0.y, fa1.y, fb1.y};
        if (need_mask) {
          const int key0 = k0 + 16 * t + 4 * s;
          const uint32_t ma0 = (key0 + 0 < valid_a ? 0xFFFFu : 0u) | (key0 + 1 < valid_a ? 0xFFFF0000u : 0u);
          const uint32_t ma1 = (key0 + 2 < valid_a ? 0xFFFFu : 0u) | (key0 + 3 < valid_a ? 0xFFFF0000u : 0u);
          const uint32_t mb0 = (key0 + 0 < valid_b ? 0xFFFFu : 0u) | (key0 + 1 < valid_b ? 0xFFFF0000u : 0u);
          const uint32_t mb1 = (key0 + 2 < valid_b ? 0xFFFFu : 0u) | (key0 + 3 < valid_b ? 0xFFFF0000u : 0u);
          ae[0] &= ma0; ao[0] &= ma0; ae[1] &= mb0; ao[1] &= mb0;
          ae[2] &= ma1; ao[2] &= ma1; ae[3] &= mb1; ao[3] &= mb1;
        }
        // V fragments: lane supplies the row address of matrix (lane / 8), row (lane % 8)
        const int mi = lane >> 3, r = lane & 7;
        const int klog = (mi & 1) * 8 + r;                                  // logical k of this address
        const int kr = (k0 - kv0) + 16 * ((klog & 7) >> 1) + 4 * s + ((klog >> 3) << 1) + (klog & 1);
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {                                    // pairs of 8-column blocks
          uint32_t b[4];
          ldmatrix_x4_trans(b, &sV[kr * kVStride + cg * 64 + jp * 16 + (mi >> 1) * 8]);
          mma_bf16(acc_e[2 * jp], ae, b[0], b[1]);
          mma_bf16(acc_o[2 * jp], ao, b[0], b[1]);
          mma_bf16(acc_e[2 * jp + 1], ae, b[2], b[3]);
          mma_bf16(acc_o[2 * jp + 1], ao, b[2], b[3]);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) { ca[i] = na[i]; cb[i] = nb[i]; }
    }
  }

  // ---- epilogue
  const float kSqrt2 = 1.41421356237309504880f;
  const float zo_lo = float(-P.zo), zo_hi = float(P.qmax - P.zo);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = h ? row_b : row_a;
    const bool row_ok = row < P.Lq;
    int code_sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = cg * 64 + j * 8 + 2 * t;
      float v[2];
      int q[2] = {0, 0};
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        v[e] = P.scale * fmaf(kSqrt2, acc_o[j][2 * h + e], acc_e[j][2 * h + e]);
        if (P.out_kind == REPQ_OUT_CODES && col + e < P.d_h && row_ok) {
          float tq = fminf(fmaxf(v[e] * P.inv_so, zo_lo), zo_hi);
          q[e] = __float2int_rn(tq) + P.zo;
          code_sum += q[e];
        }
      }
      if (row_ok && col < P.d_h) {
        const bool two = col + 1 < P.d_h;
        const int64_t roff = bo * P.o_so + bi * P.o_si + int64_t(row) * P.ldo;
        if (P.out_kind == REPQ_OUT_F32) {
          float* o = static_cast<float*>(P.out) + roff + col;
          o[0] = v[0]; if (two) o[1] = v[1];
        } else if (P.out_kind == REPQ_OUT_BF16) {
          __nv_bfloat16* o = static_cast<__nv_bfloat16*>(P.out) + roff + col;
          o[0] = __float2bfloat16_rn(v[0]); if (two) o[1] = __float2bfloat16_rn(v[1]);
        } else if (P.pack4) {
          static_cast<uint8_t*>(P.out)[roff + (col >> 1)] = uint8_t(q[0] | (q[1] << 4));
        } else {
          uint8_t* o = static_cast<uint8_t*>(P.out) + roff + col;
          o[0] = uint8_t(q[0]); if (two) o[1] = uint8_t(q[1]);
        }
      }
    }
    if (P.out_row_sum != nullptr && P.out_kind == REPQ_OUT_CODES) {
      code_sum += __shfl_xor_sync(0xffffffffu, code_sum, 1);
      code_sum += __shfl_xor_sync(0xffffffffu, code_sum, 2);
      if (t == 0 && row_ok) atomicAdd(P.out_row_sum + int64_t(bo) * P.Lq + row, code_sum);
    }
  }
}

template <int NG, bool kP4>
repq_status launch_pv(const PvParams& P, int64_t pairs, cudaStream_t st) {
  constexpr int kQRows = 16 * (8 / NG);
  constexpr size_t smem = size_t(kVKeys) * (64 * NG + 8) * sizeof(__nv_bfloat16);
  if (smem + 2048 > 48 * 1024)
    REPQ_CUDA(cudaFuncSetAttribute(pv_kernel<NG, kP4>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  dim3 grid((P.Lq + kQRows - 1) / kQRows, unsigned(pairs));
  pv_kernel<NG, kP4><<<grid, kThreads, smem, st>>>(P);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_pv(const repq_pv_desc* d, void* stream) {
  REPQ_REQUIRE(d, REPQ_INVALID_ARG, "pv: NULL descriptor");
  REPQ_REQUIRE(d->batch_outer > 0 && d->batch_inner > 0 && d->Lq >= 0 && d->Lk > 0 && d->d_h > 0, REPQ_INVALID_ARG, "pv: bad sizes");
  if (d->Lq == 0) return REPQ_OK;
  REPQ_REQUIRE(d->p_codes && d->v_codes && d->out, REPQ_INVALID_ARG, "pv: NULL pointer");
  REPQ_REQUIRE(bits_ok(d->bits_p) && bits_ok(d->bits_v), REPQ_INVALID_ARG, "pv: bits must be 4, 6 or 8");
  REPQ_REQUIRE(d->d_h % 16 == 0 && d->d_h <= 128, REPQ_UNSUPPORTED, "pv: d_h = %d must be a multiple of 16, at most 128", d->d_h);
  REPQ_REQUIRE(d->s_p > 0.f && d->s_v > 0.f, REPQ_INVALID_ARG, "pv: scales must be positive");
  REPQ_REQUIRE(aligned(d->p_codes, 16) && d->ldp_bytes % 16 == 0 && d->p_stride_pair % 16 == 0, REPQ_ALIGNMENT,
               "pv: p rows must be 16-byte aligned");
  REPQ_REQUIRE(d->ldp_bytes >= code_row_bytes(d->Lk, d->bits_p), REPQ_INVALID_ARG, "pv: ldp_bytes shorter than a row");
  REPQ_REQUIRE(d->ldv_bytes >= code_row_bytes(d->d_h, d->bits_v), REPQ_INVALID_ARG, "pv: ldv_bytes shorter than a row");
  const int qmax_v = code_max(d->bits_v);
  REPQ_REQUIRE(d->z_v >= qmax_v - 256 && d->z_v <= 256, REPQ_UNSUPPORTED,
               "pv: z_v = %d puts v - z_v outside the exactly representable range [-256, 256]", d->z_v);
  REPQ_REQUIRE(!d->causal || d->Lk >= d->Lq, REPQ_INVALID_ARG, "pv: causal needs Lk >= Lq");
  REPQ_REQUIRE(d->out_kind == REPQ_OUT_F32 || d->out_kind == REPQ_OUT_BF16 || d->out_kind == REPQ_OUT_CODES, REPQ_INVALID_ARG, "pv: unknown out_kind");
  REPQ_REQUIRE(aligned(d->out, d->out_kind == REPQ_OUT_F32 ? 4 : d->out_kind == REPQ_OUT_BF16 ? 2 : 1), REPQ_ALIGNMENT,
               "pv: out is not element-aligned");
  const int64_t pairs = int64_t(d->batch_outer) * d->batch_inner;
  REPQ_REQUIRE(pairs <= 65535, REPQ_UNSUPPORTED, "pv: more than 65535 (batch, head) pairs");
  PvParams P{};
  P.p = d->p_codes; P.bits_p = d->bits_p; P.ldp = d->ldp_bytes; P.p_pair = d->p_stride_pair;
  P.v = d->v_codes; P.bits_v = packed4(d->bits_v) ? 4 : 8; P.ldv = d->ldv_bytes; P.v_so = d->v_stride_outer; P.v_si = d->v_stride_inner;
  P.Lq = d->Lq; P.Lk = d->Lk; P.d_h = d->d_h; P.batch_inner = d->batch_inner; P.causal = d->causal;
  P.z_v = d->z_v; P.scale = d->s_p * d->s_v;
  P.out_kind = d->out_kind;
  if (d->out_kind == REPQ_OUT_CODES) {
    REPQ_REQUIRE(bits_ok(d->out_bits) && d->out_scale > 0.f, REPQ_INVALID_ARG, "pv: bad output quantizer");
    REPQ_REQUIRE(d->out_zero > -(1 << 20) && d->out_zero < (1 << 20), REPQ_INVALID_ARG, "pv: |out_zero| must be below 2^20");
    P.qmax = code_max(d->out_bits); P.pack4 = packed4(d->out_bits); P.inv_so = 1.f / d->out_scale; P.zo = d->out_zero;
  }
  P.out = d->out; P.ldo = d->ldo; P.o_so = d->o_stride_outer; P.o_si = d->o_stride_inner;
  P.out_row_sum = d->out_kind == REPQ_OUT_CODES ? d->out_row_sum : nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (pv_tc_supported(*d)) return launch_pv_tc(*d, P, st);
  const bool p4 = packed4(d->bits_p);
  if (d->d_h <= 64) return p4 ? launch_pv<1, true>(P, pairs, st) : launch_pv<1, false>(P, pairs, st);
  return p4 ? launch_pv<2, true>(P, pairs, st) : launch_pv<2, false>(P, pairs, st);
}
