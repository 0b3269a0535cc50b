/*
 * repq.h — C ABI of the RepQuant (arXiv 2402.05628) reparameterized quantized-inference hot path
 * for NVIDIA B200 (sm_100a).
 *
 * The library evaluates the *inference process* of the paper: after scale reparameterization
 * (Sec. III-C) every activation quantizer is a simple one — layer-wise uniform (Eqs. 4-5) for
 * LayerNorm outputs and all other GEMM inputs, log2 with a parity-selected scale (Eqs. 15-17) for
 * Softmax outputs — and every GEMM runs on integer codes.
 *
 * Conventions
 *  - Every entry point returns a repq_status; 0 is success.  Nothing throws, aborts or prints.
 *    repq_last_error() returns the message of the calling thread's last failure.
 *  - Pointers marked [device] are caller-owned CUDA device pointers; [host] are host pointers.
 *    The device entry points allocate no device memory: scratch comes from the `workspace` argument,
 *    sized by the matching *_workspace_bytes() call.
 *  - Device work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream) and
 *    the call returns without synchronising.
 *  - Codes are unsigned integers in [0, 2^b - 1] exactly as Eq. 4 produces them.  4-bit codes are
 *    packed two per byte (even index in the low nibble); 6- and 8-bit codes take one byte each.
 *    Every `bits` argument or field may carry the flag REPQ_BYTE_CODES (e.g. 4 | REPQ_BYTE_CODES): the
 *    quantizer is unchanged, but its codes are stored one per byte.  That is the operand format of
 *    the 8-bit integer tensor-core instruction, so 4-bit tensors kept this way need no expansion pass
 *    before a GEMM; the packed form is for storage and interchange.  Weight codes of 6 bits may also be
 *    stored four to three bytes (REPQ_PACKED6); the GEMM expands packed weight tiles in shared memory.
 *    Code tensors are row-major with a row stride in BYTES; float tensors use strides in ELEMENTS.
 *  - Weights are stored [out features j, in features c] (row j is the paper's column W[:, j]).
 *  - Zero-points are plain integers of any sign (Eq. 6 does not bound them).
 */
#ifndef REPQ_H_
#define REPQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int repq_status;
#define REPQ_OK 0
#define REPQ_INVALID_ARG 1          /* NULL pointer, non-positive size, bits not in {4,6,8}, ... */
#define REPQ_UNSUPPORTED 2          /* a size or combination the kernels do not cover */
#define REPQ_ALIGNMENT 3            /* a pointer or stride violates the stated alignment */
#define REPQ_WORKSPACE_TOO_SMALL 4
#define REPQ_CUDA_ERROR 5           /* a CUDA runtime / driver call failed (message has the detail) */
#define REPQ_TIMEOUT 6              /* a bounded device-side wait ran out (see repq_device_status) */

#define REPQ_F32 0
#define REPQ_BF16 1

#define REPQ_NORM_LAYERNORM 0
#define REPQ_NORM_RMS 1             /* mean-free variant: E[x] := 0, Var := E[x^2] */

#define REPQ_OUT_F32 0
#define REPQ_OUT_BF16 1
#define REPQ_OUT_CODES 2            /* re-quantize with Eq. 4 into `out_bits` codes */

#define REPQ_MAX_OUT_GROUPS 4

#define REPQ_BYTE_CODES 0x100       /* OR into a `bits` value: one code per byte whatever the bit width */
#define REPQ_PACKED6 0x200          /* 6 | REPQ_PACKED6, weight codes only (repq_pack_weights, the weight operand of a
                                       plain repq_qgemm, repq_block_desc.bits_w): four codes in three bytes, code i of
                                       a row in bits [6i, 6i + 6) of the row read as a little-endian bit string */

/* Copies the calling thread's last error message (NUL-terminated, truncated to n) and returns its
 * full length. */
size_t repq_last_error(char* buf, size_t n);

/* Library ABI version (bumped on any signature change). */
int repq_abi_version(void);   /* currently 5 */

/* ------------------------------------------------------------------------------------------------
 * One-time host-side preparation (not on the timed path)
 * ---------------------------------------------------------------------------------------------- */

/* Eq. 6: s = (x_up - x_low) / (2^b - 1) rounded to float32, z = round(-x_low / s), for n independent
 * quantizers (n = D for channel-wise, n = 1 for layer-wise).  All pointers [host]. */
repq_status repq_scale_zero_from_bounds(int n, const float* x_low, const float* x_up, int bits,
                                        float* s, int32_t* z);

/* Scale reparameterization for LayerNorm activations, Eqs. 10-14 (Sec. III-C.1).
 * In  [host]: gamma, beta, s (float[D]), z (int32[D]) — LayerNorm affine factors and the channel-wise
 *             quantizer; W (float N x D, row-major, dense), b (float[N] or NULL) — the next layer.
 * Out [host]: gamma_t, beta_t (float[D]) = gamma / r1, (beta + s*r2) / r1; *s_t = mean(s);
 *             *z_t = mean(z) rounded half-to-even to an integer (so r2 = z - z_t is integral, as
 *             Eq. 10 needs); W_t (N x D) = W * r1 per input channel; b_t (float[N]) = b - W (s*r2).
 * Arithmetic is float64, results rounded once to float32.  W_t may alias W; b_t may alias b. */
repq_status repq_fold_ln(int D, int N, const float* gamma, const float* beta, const float* s,
                         const int32_t* z, const float* W, const float* b, float* gamma_t,
                         float* beta_t, float* s_t, int32_t* z_t, float* W_t, float* b_t);

/* Channel-wise (per output feature) round-to-nearest weight quantization, Eqs. 4-6; bounds per row
 * are min(row, 0) and max(row, 0) so that 0 <= z_w <= 2^b - 1; an all-zero row gets s_w = 1.
 * In  [host]: W (float N x K, row-major, dense).
 * Out [host]: codes (N rows of ld_codes_bytes bytes; ld_codes_bytes >= K*bits/8 rounded up, multiple
 *             of 16; bits_w may carry REPQ_BYTE_CODES, or be 6 | REPQ_PACKED6), s_w (float[N]), z_w (int32[N]),
 *             w_row_sum (int32[N]) = sum_c codes[j, c]. */
repq_status repq_pack_weights(int N, int K, int bits_w, const float* W, uint8_t* codes,
                              int64_t ld_codes_bytes, float* s_w, int32_t* z_w, int32_t* w_row_sum);

/* Full-precision normalisation (Eq. 9; REPQ_NORM_RMS: the mean-free variant) of a calibration batch, float32 out:
 * the activations X' that repq_dual_clip learns its clipping factors on.  Calibration-time only; the inference
 * path (repq_ln_quant) never forms X'.  x [device]: rows x D, REPQ_F32 or REPQ_BF16, row stride ldx elements;
 * gamma, beta [device] float[D] (the un-reparameterized affine factors); y [device]: rows x D float32, row stride ldy. */
repq_status repq_layernorm(const void* x, int x_dtype, int64_t rows, int D, int64_t ldx, const float* gamma,
                           const float* beta, float eps, int norm_kind, float* y, int64_t ldy, void* stream);

/* Per-channel dual clipping (Sec. III-D, Eqs. 18-20): the clipping bounds of the channel-wise quantizer of a
 * LayerNorm activation, learned on a calibration batch just before the scale reparameterization
 * (repq_scale_zero_from_bounds -> repq_fold_ln take them from here).  For every channel d
 *     x_up[d] = max_d sigmoid(alpha1_d),   x_low[d] = min_d sigmoid(alpha2_d)                   (Eqs. 18-19)
 * with the factors found by `iters` Adam steps of size `lr` (Sec. IV-A: 100 steps of 0.01; decay rates 0.9 / 0.999,
 * epsilon 1e-8) on || X'_{:,d} - X^'_{:,d} ||^2 (Eq. 20), X^' = Eq. 5 of Eq. 4 with the (s, z) of Eq. 6 on those
 * bounds; the round operations pass the gradient straight through, the clip passes it on [0, 2^bits - 1].
 * `alpha0` is the factors' starting value (the paper gives none; 0 starts at half of the extremes).
 * x [device]: n x D float32 activations, row stride ldx elements.  x_low, x_up [device] float[D].
 * loss [device] double[2 D] or NULL: the objective per channel before the first step and with the returned
 * bounds.  A channel whose contracted extremes coincide (a constant channel) is left alone: its factors keep alpha0,
 * its objective reads 0 and x_low = x_up is returned (Eq. 6 has no scale for it; the caller decides).  Runs in float64 on `stream`, one kernel, no scratch memory; channels are independent. */
repq_status repq_dual_clip(const float* x, int64_t n, int D, int64_t ldx, int bits, int iters, float lr,
                           float alpha0, float* x_low, float* x_up, double* loss, void* stream);

/* Rotation table of the rotary position embedding for repq_gemm_desc.rope_cos_sin.  (The paper's block,
 * Eqs. 1-3, has no position embedding inside; the LLaMA models it evaluates in Sec. IV-A rotate Q and K.)
 * table [host]: seq x (d_h / 2) pairs of floats, table[(m * d_h / 2 + i) * 2 + {0, 1}] = cos, sin of
 * m * base^(-2 i / d_h), evaluated in float64 and rounded once.  d_h must be even. */
repq_status repq_rope_table(int seq, int d_h, double base, float* table);

/* ------------------------------------------------------------------------------------------------
 * Hot path, stage by stage
 * ---------------------------------------------------------------------------------------------- */

/* LayerNorm (Eq. 9) with the reparameterized affine factors (Eq. 12), followed by layer-wise uniform
 * quantization (Eq. 4) with the scalar (s_t, z_t):
 *     y = (x - E[x]) / sqrt(Var[x] + eps) * gamma_t + beta_t   per row, population variance
 *     q = clip(round(y / s_t) + z_t, 0, 2^bits - 1)            round = half to even
 * x [device]: rows x D, dtype REPQ_F32 or REPQ_BF16, row stride ldx elements; x and ldx must keep every
 *   row 16-byte aligned.  D must be a multiple of 8 and at most 16384.
 * gamma_t, beta_t [device] float[D].  codes [device]: rows of ld_codes_bytes bytes (4-bit: multiple of
 *   4; 6/8-bit: multiple of 8).  row_sum [device] int32[rows] or NULL: sum of the row's codes (the
 *   activation term of the GEMM's zero-point correction). */
repq_status repq_ln_quant(const void* x, int x_dtype, int64_t rows, int D, int64_t ldx,
                          const float* gamma_t, const float* beta_t, float eps, int norm_kind,
                          float s_t, int z_t, int bits, uint8_t* codes, int64_t ld_codes_bytes,
                          int32_t* row_sum, void* stream);

/* Quantized linear layer / batched code-by-code product.  Inference form of Sec. III-A (integer
 * inputs and weights of every matrix multiplication) with the compensation of Eqs. 13-14 already
 * folded into the weights and bias:
 *     acc[m, j]  = sum_c a[m, c] w[j, c]                                   (int32, exact)
 *     corr[m, j] = acc - z_w[j] asum[m] - z_a wsum[j] + K z_a z_w[j]       (= sum (a - z_a)(w - z_w))
 *     v          = alpha * s_a * s_w[j] * corr + bias[j]                   (float32)
 *     v          = gelu(v) if `gelu`;  v += residual[m, j] if `residual`
 *     out        = v (f32 / bf16)   or   clip(round(v / s_o) + z_o, 0, 2^out_bits - 1)
 * A batch of batch_outer x batch_inner independent products shares every scalar; operand (bo, bi)
 * starts at base + bo*stride_outer + bi*stride_inner. */
typedef struct repq_gemm_desc {
  int32_t M, N, K;
  int32_t batch_outer, batch_inner;     /* both 1 for a plain GEMM */
  /* activation codes a: [M, K] */
  const uint8_t* a_codes;               /* [device] */
  int32_t bits_a;                       /* 4, 6 or 8 */
  int64_t lda_bytes, a_stride_outer, a_stride_inner;    /* bytes */
  float s_a;                            /* layer-wise scale (s~ after a LayerNorm) */
  int32_t z_a;                          /* layer-wise zero-point (z~) */
  const int32_t* a_row_sum;             /* [device] int32[M], plain GEMM only; NULL = computed here */
  /* weight codes w: [N, K] */
  const uint8_t* w_codes;               /* [device] */
  int32_t bits_w;                       /* 4, 6 or 8 (| REPQ_BYTE_CODES), or 6 | REPQ_PACKED6 (plain GEMM only) */
  int64_t ldw_bytes, w_stride_outer, w_stride_inner;    /* bytes */
  const float* s_w;                     /* [device] float[N] per output channel; NULL = s_w_scalar */
  const int32_t* z_w;                   /* [device] int32[N]; NULL = z_w_scalar */
  float s_w_scalar;
  int32_t z_w_scalar;
  const int32_t* w_row_sum;             /* [device] int32[N], plain GEMM only; NULL = computed here */
  const float* bias;                    /* [device] float[N] (b~ after a LayerNorm) or NULL */
  float alpha;                          /* e.g. 1/sqrt(d_h) for attention scores; 1 otherwise */
  /* epilogue */
  int32_t gelu;                         /* erf-form GELU */
  const void* residual;                 /* [device] M x N, dtype residual_dtype, or NULL (plain GEMM) */
  int32_t residual_dtype;
  int64_t ld_residual;                  /* elements */
  int32_t out_kind;                     /* REPQ_OUT_* */
  int32_t out_bits;
  int32_t out_groups;                   /* 1..4: output columns split into equal ranges, each with its
                                           own (s_o, z_o) — e.g. 3 for a fused Q|K|V projection */
  float out_scale[REPQ_MAX_OUT_GROUPS];
  int32_t out_zero[REPQ_MAX_OUT_GROUPS];
  void* out;                            /* [device] */
  int64_t ldo, o_stride_outer, o_stride_inner;          /* elements (float kinds) or bytes (codes) */
  int32_t* out_row_sum;                 /* [device] int32[M] or NULL: with REPQ_OUT_CODES, the row sums
                                           of the produced codes are ADDED here (caller zero-fills) */
  int32_t* acc_debug;                   /* [device] int32 M x N (dense) raw accumulators, or NULL */
  int32_t causal;                       /* != 0: outputs with n > m + (N - M) are never read by the caller
                                           and may be left unwritten (attention scores under a causal mask) */
  /* Two optional steps between v and the output conversion, on pairs of neighbouring output columns (plain GEMM
   * only, not together with gelu or residual).  Neither is part of the paper's block (Eqs. 1-3); they serve the
   * LLaMA block form of the models in Sec. IV-A, where the quantizer of Eq. 4 follows them.
   *  - rope_cos_sin != NULL: rotary position embedding.  [device] table of repq_rope_table for rope_period
   *    positions and heads of rope_dim channels (16-byte aligned).  Row m has position m mod rope_period; inside
   *    the first rope_groups of the out_groups equal column ranges (out_groups delimits the ranges in every output
   *    kind; with float outputs it has no other effect), the pair
   *    (v[2i], v[2i+1]) of every head is rotated by the angle of (position, i):
   *        v'[2i] = v[2i] cos - v[2i+1] sin,   v'[2i+1] = v[2i] sin + v[2i+1] cos.
   *    rope_dim must be a multiple of 16 and divide N / out_groups.
   *  - glu != 0: gated linear unit.  Weight rows (2i, 2i+1) are (gate_i, up_i); the output has N / 2 columns,
   *    out[m, i] = silu(v[m, 2i]) * v[m, 2i+1], silu(x) = x / (1 + exp(-x)); ldo, out_groups and the output
   *    quantizer refer to those N / 2 columns.  N must be even. */
  const float* rope_cos_sin;
  int32_t rope_period, rope_dim, rope_groups;
  int32_t glu;
} repq_gemm_desc;

repq_status repq_qgemm_workspace_bytes(const repq_gemm_desc* d, size_t* bytes);
repq_status repq_qgemm(const repq_gemm_desc* d, void* workspace, size_t workspace_bytes, void* stream);

/* Softmax (Eq. 3) over each row of `scores`, then the log-sqrt2 quantizer in its base-2 form
 * (Eq. 15, second line):  A = softmax(pre_scale * scores_row);
 *     p = clip(round(-2 log2(A / s)), 0, 2^bits - 1).
 * scores [device]: rows x L, REPQ_F32 or REPQ_BF16, row stride ld elements; the buffer holds rows x ld elements
 * and the padding [L, ld) of a row may be read (its values are ignored).  Rows that start on a 16-byte boundary
 * with a 16-byte multiple stride take the fast kernels.
 * Causal masking is structural: if causal_period > 0, row r sees only its first
 *     min(L, (r mod causal_period) + 1 + causal_offset) keys;
 * codes of masked keys are written as 2^bits - 1 and must not be read as probabilities.
 * codes [device]: rows of ld_codes_bytes bytes (multiple of 4).  s > 0 is the log-sqrt2 scale. */
repq_status repq_softmax_log2(const void* scores, int dtype, int64_t rows, int L, int64_t ld,
                              float pre_scale, int causal_period, int causal_offset, float s, int bits,
                              uint8_t* codes, int64_t ld_codes_bytes, void* stream);

/* P.V with Softmax codes de-quantized by the reparameterized log2 rule (Eqs. 16-17):
 *     A^[i, j] = s * 2^(-ceil(p/2)) * (sqrt2 if p odd else 1)
 *     O[i, :]  = sum_j A^[i, j] * s_v * (v[j, :] - z_v)          (causal: j <= i + Lk - Lq only)
 * for batch_outer x batch_inner (batch, head) pairs.  p [device]: per pair an Lq x Lk code matrix,
 * row stride ldp_bytes, pair (bo, bi) at p + (bo*batch_inner + bi) * p_stride_pair bytes.
 * v [device]: Lk x d_h codes, row stride ldv_bytes, pair at v + bo*v_stride_outer + bi*v_stride_inner.
 * The output uses the same epilogue kinds as repq_qgemm (one group).  d_h must be a multiple of 16, at
 * most 128. */
typedef struct repq_pv_desc {
  int32_t batch_outer, batch_inner, Lq, Lk, d_h;
  const uint8_t* p_codes;
  int32_t bits_p;
  int64_t ldp_bytes, p_stride_pair;
  float s_p;                            /* log-sqrt2 scale s */
  const uint8_t* v_codes;
  int32_t bits_v;
  int64_t ldv_bytes, v_stride_outer, v_stride_inner;
  float s_v;
  int32_t z_v;
  int32_t causal;
  int32_t out_kind, out_bits;
  float out_scale;
  int32_t out_zero;
  void* out;
  int64_t ldo, o_stride_outer, o_stride_inner;
  int32_t* out_row_sum;                 /* as in repq_gemm_desc; rows are indexed bo*Lq + i */
} repq_pv_desc;

repq_status repq_pv(const repq_pv_desc* d, void* stream);

/* Fused attention on codes: Eq. 3 (scores from quantized Q and K, Softmax), Eq. 15 (log-sqrt2 codes of the
 * probabilities) and Eqs. 16-17 (P.V with the reparameterized log2 de-quantization) in one kernel; scores and
 * codes stay on chip.  Same result as repq_qgemm (scores) -> repq_softmax_log2 -> repq_pv, except that the
 * Softmax sum is accumulated in a different order, which can move a code across a rounding tie.
 *     S[i, j] = alpha s_q s_k sum_c (q[i, c] - z_q)(k[j, c] - z_k)      (causal: j <= i + Lk - Lq only)
 *     p       = clip(round(-2 log2(softmax(S)[i, j] / s_p)), 0, 2^bits_p - 1)
 *     O[i, :] = sum_j s_p 2^(-ceil(p/2)) (sqrt2 if p odd) s_v (v[j, :] - z_v)
 * for batch_outer x batch_inner (batch, head) pairs.  q, k, v [device]: codes of one quantizer width, stored one
 * per byte (bits_qkv must carry REPQ_BYTE_CODES); operand (bo, bi) starts at base + bo*stride_outer +
 * bi*stride_inner; Q and K rows 16-byte aligned, V rows 8-byte aligned.  d_h a multiple of 16, at most 128.
 * Output as in repq_pv.
 * For 4-bit Q / K quantizers with 0 <= z_q <= 15 the score contraction runs on the tensor cores' 8-bit float type
 * (the operands are integers of at most 15 in magnitude, exactly representable; products and sums are exact in the
 * float32 accumulator), which saves the integer -> float conversion of every score; the result is bit-identical to
 * the integer contraction, which the environment variable REPQ_ATTENTION_INT_SCORES=1 (read at every call) selects
 * instead. */
typedef struct repq_attention_desc {
  int32_t batch_outer, batch_inner, Lq, Lk, d_h;
  int32_t bits_qkv;
  const uint8_t* q_codes;
  int64_t ldq_bytes, q_stride_outer, q_stride_inner;
  float s_q;
  int32_t z_q;
  const uint8_t* k_codes;
  int64_t ldk_bytes, k_stride_outer, k_stride_inner;
  float s_k;
  int32_t z_k;
  const uint8_t* v_codes;
  int64_t ldv_bytes, v_stride_outer, v_stride_inner;
  float s_v;
  int32_t z_v;
  float alpha;                          /* 1/sqrt(d_h) */
  int32_t causal;
  int32_t bits_p;                       /* width of the log-sqrt2 quantizer */
  float s_p;                            /* its scale s */
  int32_t out_kind, out_bits;
  float out_scale;
  int32_t out_zero;
  void* out;
  int64_t ldo, o_stride_outer, o_stride_inner;
  int32_t* out_row_sum;                 /* as in repq_pv_desc */
} repq_attention_desc;

repq_status repq_attention(const repq_attention_desc* d, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Whole block: Eqs. 1-2,  X_bar = MSA(LN(X)) + X,  Y = MLP(LN(X_bar)) + X_bar, all GEMM inputs
 * quantized (LayerNorm -> QKV -> QK^T -> Softmax/log2 -> P.V -> proj -> LayerNorm -> fc1/GELU -> fc2).
 *
 * Besides the paper's own block form, the LLaMA form of the models of Sec. IV-A (which the paper evaluates
 * but does not write down) is selected by three independent fields: norm_kind = REPQ_NORM_RMS (mean-free
 * normalisation; its channel-wise quantizer is reparameterized by Eqs. 10-14 like LayerNorm's, so gamma_t
 * and beta_t are both used), rope != 0 (Q and K of the projection are rotated by the table in
 * repq_block_params.rope_cos_sin before their quantizers) and mlp_kind = REPQ_MLP_SWIGLU
 * (Y = down(silu(gate(.)) * up(.)) + X_bar: `fc1` then holds 2*mlp weight rows, gate_i and up_i
 * interleaved as rows 2i and 2i+1, and `fc2` is the down projection).
 * ---------------------------------------------------------------------------------------------- */
#define REPQ_MLP_GELU 0
#define REPQ_MLP_SWIGLU 1
typedef struct repq_linear_params {
  const uint8_t* w_codes;               /* [device] packed by repq_pack_weights */
  int64_t ldw_bytes;
  const float* s_w;                     /* [device] float[N] */
  const int32_t* z_w;                   /* [device] int32[N] */
  const int32_t* w_row_sum;             /* [device] int32[N] */
  const float* bias;                    /* [device] float[N] */
} repq_linear_params;

typedef struct repq_block_desc {
  int32_t batch, seq, dim, heads, mlp;
  int32_t bits_a, bits_w, bits_p;       /* bits_w describes the layout of the w_codes given (it may carry
                                           REPQ_BYTE_CODES); activation codes are internal and byte-wide */
  int32_t causal;
  int32_t norm_kind;
  float eps;
  int32_t act_dtype;                    /* dtype of x and of the stored residual stream X_bar */
  int32_t out_dtype;                    /* dtype of y */
  int32_t staged_attention;             /* 0: fused attention kernel (repq_attention); != 0: the three separate
                                           stages (scores -> Softmax codes -> P.V) through the workspace */
  int32_t rope;                         /* != 0: rotary position embedding on Q and K (position = token index) */
  int32_t mlp_kind;                     /* REPQ_MLP_GELU (the paper's block) or REPQ_MLP_SWIGLU */
} repq_block_desc;

typedef struct repq_block_params {
  const float* ln1_gamma_t;             /* [device] folded LayerNorm-1 factors */
  const float* ln1_beta_t;
  float ln1_s;
  int32_t ln1_z;
  repq_linear_params qkv;               /* N = 3*dim (q | k | v), K = dim, weights W~ */
  float s_q, s_k, s_v;
  int32_t z_q, z_k, z_v;
  float softmax_s;                      /* log-sqrt2 scale */
  float s_attn;
  int32_t z_attn;                       /* quantizer of the attention output (input of proj) */
  repq_linear_params proj;              /* N = K = dim */
  const float* ln2_gamma_t;
  const float* ln2_beta_t;
  float ln2_s;
  int32_t ln2_z;
  repq_linear_params fc1;               /* N = mlp (REPQ_MLP_SWIGLU: 2*mlp, gate / up interleaved), K = dim, weights W~ */
  float s_hidden;
  int32_t z_hidden;                     /* quantizer of the GELU output (input of fc2) */
  repq_linear_params fc2;               /* N = dim, K = mlp */
  const float* rope_cos_sin;            /* [device] repq_rope_table(seq, dim / heads, base), or NULL if !rope */
} repq_block_params;

repq_status repq_block_workspace_bytes(const repq_block_desc* d, size_t* bytes);

/* x [device]: (batch*seq) x dim, dense, dtype act_dtype.  y [device]: same shape, dtype out_dtype. */
repq_status repq_block_forward(const repq_block_desc* d, const repq_block_params* p, const void* x,
                               void* y, void* workspace, size_t workspace_bytes, void* stream);

/* Number of stages repq_block_forward runs, and a variant of it that also measures them: CUDA events are
 * recorded on `stream` between the stages, the call synchronises the stream and writes the duration
 * of each stage in milliseconds to stage_ms [host, REPQ_BLOCK_STAGES floats], in the order
 * ln1, qkv, scores, softmax, pv, proj, ln2, fc1, fc2.  Same results as repq_block_forward.
 * (Measurement aid: the paper has no counterpart.) */
#define REPQ_BLOCK_STAGES 9
repq_status repq_block_forward_timed(const repq_block_desc* d, const repq_block_params* p, const void* x,
                                     void* y, void* workspace, size_t workspace_bytes, void* stream,
                                     float* stage_ms);

/* repq_block_forward for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a deployment convenience.)
 *
 * Some hosts of this library never get to call cudaMalloc on the inference path: a plug-in that runs
 * inside another runtime's memory plan, a real-time serving loop whose allocator is frozen after
 * start-up, a sandbox that hands out device pointers but not the allocator.  Those callers still pass
 * x, y and the parameter block as usual, but give no workspace: the intermediates of the block live in
 * a scratch array that is part of the library image itself (a file-scope __device__ array of
 * REPQ_STATIC_WORKSPACE_BYTES, 8 MiB, resident on every GPU that loads the library until the process
 * exits).  The call allocates nothing: no cudaMalloc / cudaFree, no allocating library routine.
 *
 *  - Size limit: the block must need at most REPQ_STATIC_WORKSPACE_BYTES of workspace
 *    (repq_block_workspace_bytes tells; a ViT-S-sized block of a few hundred tokens fits).  Larger
 *    blocks are rejected with REPQ_WORKSPACE_TOO_SMALL and a message naming both sizes.
 *  - First call on a device: the library looks up the device address of its scratch array once per
 *    device (with that device current) and remembers it (threads that race on that first call both
 *    look it up and store the same address).  Make that first call outside any stream capture.
 *  - The scratch is shared by every call in the process and keeps whatever the previous call left in
 *    it; the entry point itself clears the parts that have to start at zero.  Two calls that overlap
 *    in time on the same GPU (different streams or threads) race on it: serialise them.
 * Results are identical to repq_block_forward with a caller-provided workspace. */
#define REPQ_STATIC_WORKSPACE_BYTES (8u << 20)
repq_status repq_block_forward_static(const repq_block_desc* d, const repq_block_params* p, const void* x,
                                      void* y, void* stream);

/* repq_block_forward for a sequence of n_batches independent batches whose inputs and outputs are in HOST
 * memory: batch i is read from x_host[i] and its result written to y_host[i] (each (batch*seq) x dim, dense,
 * act_dtype / out_dtype).  The library copies through the caller's device staging buffers and overlaps the
 * copies with the block's kernels: batch i + 1 is copied in and batch i - 1 copied out while batch i is
 * computed (two helper streams per device, created on first use and kept).  The same x_host or y_host pointer
 * may be given for several batches.  (Plumbing around Eqs. 1-3 of the block; the paper has no counterpart.)
 *
 *  - x_dev[2], y_dev[2] [device]: staging buffers of one batch each; workspace as for repq_block_forward
 *    (one suffices: the blocks themselves run one after the other on `stream`).  Owned by the caller, who
 *    may not touch them until `stream` has completed.
 *  - Host buffers should be page-locked: with pageable memory the copies are correct but do not overlap.
 *  - Ordering: everything is queued after the work already on `stream`; the call returns when the work is
 *    queued, and `stream` completes after the last copy out, so synchronising `stream` (or an event recorded
 *    on it) makes every y_host[i] valid.  Two calls that overlap in time on the same device must use
 *    different staging buffers and are serialised on the helper streams.
 *  - Errors: REPQ_INVALID_ARG for NULL pointers or staging buffers that alias; errors of repq_block_forward
 *    are passed on (work queued before the error still runs). */
typedef struct repq_host_staging {
  void* x_dev[2];
  void* y_dev[2];
  void* workspace;
  size_t workspace_bytes;
} repq_host_staging;
repq_status repq_block_forward_host(const repq_block_desc* d, const repq_block_params* p,
                                    const void* const* x_host, void* const* y_host, int n_batches,
                                    const repq_host_staging* s, void* stream);

/* Number of CUDA kernels this library has launched in the calling process so far. */
uint64_t repq_launch_count(void);

/* Device-side health word of the calling thread's current device: 0 = healthy; non-zero = a bounded
 * wait inside a kernel gave up (the kernel drained and returned; results of that launch are
 * invalid).  Synchronises the device and writes the word to *status; returns REPQ_OK if it is 0 and
 * REPQ_TIMEOUT otherwise.  `reset` != 0 clears it. */
repq_status repq_device_status(int32_t* status, int reset);

/* Self-test of the failure path of the bounded device-side waits.  (Every mbarrier wait of the
 * tensor-core kernels gives up after about a second, records a code in the health word and lets the kernel
 * drain and return instead of hanging; the paper has no counterpart.)  Launches, on `stream`, a one-thread
 * kernel whose barrier is never completed and whose wait uses the same routine with a limit of
 * limit_cycles SM clock cycles (1 .. 2e9): the kernel returns after that long, repq_device_status then
 * reports REPQ_TIMEOUT with code 77 until it is reset, and the context stays usable. */
repq_status repq_bounded_wait_selftest(int64_t limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* REPQ_H_ */
