// repq_block_forward: one quantized transformer block (Eqs. 1-3) as a stream-ordered sequence of the
// stage kernels.  No host synchronisation, no allocation: every intermediate lives in the caller's
// workspace.
#include <atomic>
#include <cmath>

#include "kernels.h"

namespace repq {
namespace {

struct BlockLayout {
  int64_t M, ld_a, ld_qkv, ld_s, ld_p, ld_h;
  size_t off_ln, off_asum, off_qkv, off_scores, off_p, off_attn, off_asum_attn, off_xbar, off_hidden,
      off_asum_h, off_gemm_ws, gemm_ws, total;
};

inline size_t bump(size_t& cur, size_t bytes) {
  const size_t at = cur;
  cur += (bytes + 255) / 256 * 256;
  return at;
}

repq_status validate(const repq_block_desc& d) {
  REPQ_REQUIRE(d.batch > 0 && d.seq > 0 && d.dim > 0 && d.heads > 0 && d.mlp > 0, REPQ_INVALID_ARG, "block: sizes must be positive");
  REPQ_REQUIRE(d.dim % d.heads == 0, REPQ_INVALID_ARG, "block: dim must be a multiple of heads");
  REPQ_REQUIRE(bits_ok(d.bits_a) && bits_w_ok(d.bits_w) && bits_ok(d.bits_p), REPQ_INVALID_ARG, "block: bits must be 4, 6 or 8");
  REPQ_REQUIRE(d.dim % 8 == 0 && d.mlp % 8 == 0, REPQ_UNSUPPORTED, "block: dim and mlp must be multiples of 8");
  const int dh = d.dim / d.heads;
  REPQ_REQUIRE(dh % 16 == 0 && dh <= 128, REPQ_UNSUPPORTED, "block: head dim %d must be a multiple of 16, at most 128", dh);
  REPQ_REQUIRE(d.seq <= 16384, REPQ_UNSUPPORTED, "block: seq exceeds 16384");
  REPQ_REQUIRE((d.act_dtype == REPQ_F32 || d.act_dtype == REPQ_BF16) && (d.out_dtype == REPQ_F32 || d.out_dtype == REPQ_BF16),
               REPQ_INVALID_ARG, "block: dtypes must be REPQ_F32 or REPQ_BF16");
  REPQ_REQUIRE(d.norm_kind == REPQ_NORM_LAYERNORM || d.norm_kind == REPQ_NORM_RMS, REPQ_INVALID_ARG, "block: unknown norm_kind");
  REPQ_REQUIRE(int64_t(d.batch) * d.heads <= 65535, REPQ_UNSUPPORTED, "block: batch * heads exceeds 65535");
  REPQ_REQUIRE(int64_t(d.batch) * d.seq <= 2147483647LL, REPQ_UNSUPPORTED, "block: batch * seq exceeds 2^31 - 1");
  REPQ_REQUIRE(d.mlp_kind == REPQ_MLP_GELU || d.mlp_kind == REPQ_MLP_SWIGLU, REPQ_INVALID_ARG, "block: unknown mlp_kind");
  REPQ_REQUIRE(!d.rope || dh % 16 == 0, REPQ_UNSUPPORTED, "block: rope needs a head dim that is a multiple of 16");
  return REPQ_OK;
}

// Activation codes between the stages are internal to the block: they are kept one per byte, the operand
// format of the integer tensor-core instruction, whatever their bit width.
inline int act_bits(const repq_block_desc& d) { return d.bits_a | REPQ_BYTE_CODES; }

repq_gemm_desc linear_desc(const repq_block_desc& d, int64_t M, int N, int K, const uint8_t* a, int64_t lda,
                           float s_a, int z_a, const int32_t* asum, const repq_linear_params& w) {
  repq_gemm_desc g{};
  g.M = int32_t(M); g.N = N; g.K = K; g.batch_outer = g.batch_inner = 1;
  g.a_codes = a; g.bits_a = act_bits(d); g.lda_bytes = lda; g.s_a = s_a; g.z_a = z_a; g.a_row_sum = asum;
  g.w_codes = w.w_codes; g.bits_w = d.bits_w; g.ldw_bytes = w.ldw_bytes; g.s_w = w.s_w; g.z_w = w.z_w;
  g.w_row_sum = w.w_row_sum; g.bias = w.bias; g.alpha = 1.f;
  g.out_groups = 1; g.out_scale[0] = 1.f;
  return g;
}

BlockLayout layout(const repq_block_desc& d) {
  BlockLayout L{};
  L.M = int64_t(d.batch) * d.seq;
  L.ld_a = round_up(code_row_bytes(d.dim, act_bits(d)), 16);
  L.ld_qkv = round_up(code_row_bytes(3 * int64_t(d.dim), act_bits(d)), 16);
  L.ld_h = round_up(code_row_bytes(d.mlp, act_bits(d)), 16);
  L.ld_s = round_up(d.seq, 4);
  L.ld_p = round_up((int64_t(d.seq) + 7) / 8 * (d.bits_p == 4 ? 4 : 8), 16);
  const int64_t rows_s = int64_t(d.batch) * d.heads * d.seq;
  const size_t act = d.act_dtype == REPQ_F32 ? 4 : 2;
  size_t cur = 0;
  L.off_ln = bump(cur, size_t(L.M * L.ld_a));
  L.off_asum = bump(cur, size_t(L.M) * 4);
  L.off_qkv = bump(cur, size_t(L.M * L.ld_qkv));
  // float32 scores and Softmax codes exist only when the three attention stages run as separate kernels
  L.off_scores = bump(cur, d.staged_attention ? size_t(rows_s * L.ld_s) * 4 : 0);
  L.off_p = bump(cur, d.staged_attention ? size_t(rows_s * L.ld_p) : 0);
  L.off_attn = bump(cur, size_t(L.M * L.ld_a));
  L.off_asum_attn = bump(cur, size_t(L.M) * 4);
  L.off_xbar = bump(cur, size_t(L.M) * d.dim * act);
  L.off_hidden = bump(cur, size_t(L.M * L.ld_h));
  L.off_asum_h = bump(cur, size_t(L.M) * 4);
  // scratch of the largest GEMM of the block
  repq_linear_params none{};
  size_t ws = 0;
  const int n_fc1 = d.mlp_kind == REPQ_MLP_SWIGLU ? 2 * d.mlp : d.mlp;
  const int shapes[4][2] = {{3 * d.dim, d.dim}, {d.dim, d.dim}, {n_fc1, d.dim}, {d.dim, d.mlp}};
  for (auto& s : shapes) {
    repq_gemm_desc g = linear_desc(d, L.M, s[0], s[1], nullptr, code_row_bytes(s[1], act_bits(d)), 1.f, 0, nullptr, none);
    g.ldw_bytes = round_up(code_row_bytes(s[1], d.bits_w), 16);
    g.lda_bytes = round_up(code_row_bytes(s[1], act_bits(d)), 16);
    if (qgemm_tc_supported(g)) ws = ws > qgemm_tc_workspace(g) ? ws : qgemm_tc_workspace(g);
  }
  L.gemm_ws = ws;
  L.off_gemm_ws = bump(cur, ws);
  L.total = cur;
  return L;
}

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_block_workspace_bytes(const repq_block_desc* d, size_t* bytes) {
  REPQ_REQUIRE(d && bytes, REPQ_INVALID_ARG, "block_workspace_bytes: NULL argument");
  REPQ_TRY(validate(*d));
  *bytes = layout(*d).total;
  return REPQ_OK;
}

static repq_status block_forward_impl(const repq_block_desc* dp, const repq_block_params* pp, const void* x,
                                      void* y, void* workspace, size_t workspace_bytes, void* stream,
                                      cudaEvent_t* marks) {
  REPQ_REQUIRE(dp && pp && x && y, REPQ_INVALID_ARG, "block_forward: NULL argument");
  const repq_block_desc& d = *dp;
  const repq_block_params& p = *pp;
  REPQ_TRY(validate(d));
  REPQ_REQUIRE(!d.rope || p.rope_cos_sin != nullptr, REPQ_INVALID_ARG, "block_forward: rope is set but rope_cos_sin is NULL");
  const BlockLayout L = layout(d);
  REPQ_REQUIRE(workspace && workspace_bytes >= L.total, REPQ_WORKSPACE_TOO_SMALL,
               "block_forward: workspace of %zu bytes given, %zu needed", workspace_bytes, L.total);
  REPQ_REQUIRE(aligned(workspace, 256), REPQ_ALIGNMENT, "block_forward: workspace must be 256-byte aligned");
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = d.dim, H = d.heads, dh = D / H, S = d.seq;
  const int64_t M = L.M;
  const int ab = act_bits(d);
  const int64_t head_bytes = code_row_bytes(dh, ab);          // bytes of one head's codes in a row

  uint8_t* ln_c = ws + L.off_ln;
  int32_t* asum = reinterpret_cast<int32_t*>(ws + L.off_asum);
  uint8_t* qkv_c = ws + L.off_qkv;
  float* scores = reinterpret_cast<float*>(ws + L.off_scores);
  uint8_t* p_c = ws + L.off_p;
  uint8_t* attn_c = ws + L.off_attn;
  int32_t* asum_attn = reinterpret_cast<int32_t*>(ws + L.off_asum_attn);
  void* xbar = ws + L.off_xbar;
  uint8_t* hid_c = ws + L.off_hidden;
  int32_t* asum_h = reinterpret_cast<int32_t*>(ws + L.off_asum_h);
  void* gws = ws + L.off_gemm_ws;
  // the two row-sum accumulators that kernels add into start at zero; cleared here, ahead of the first kernel,
  // so that the kernels of the block follow one another in the stream without anything in between
  REPQ_CUDA(cudaMemsetAsync(asum_attn, 0, size_t(M) * 4, st));
  REPQ_CUDA(cudaMemsetAsync(asum_h, 0, size_t(M) * 4, st));
  int n_mark = 0;
#define REPQ_MARK()                                            \
  do {                                                         \
    if (marks) REPQ_CUDA(cudaEventRecord(marks[n_mark++], st)); \
  } while (0)
  REPQ_MARK();

  // ---- X_bar = MSA(LN(X)) + X
  REPQ_TRY(repq_ln_quant(x, d.act_dtype, M, D, D, p.ln1_gamma_t, p.ln1_beta_t, d.eps, d.norm_kind, p.ln1_s, p.ln1_z,
                         ab, ln_c, L.ld_a, asum, stream));
  REPQ_MARK();
  {
    repq_gemm_desc g = linear_desc(d, M, 3 * D, D, ln_c, L.ld_a, p.ln1_s, p.ln1_z, asum, p.qkv);
    g.out_kind = REPQ_OUT_CODES; g.out_bits = ab; g.out_groups = 3;
    g.out_scale[0] = p.s_q; g.out_scale[1] = p.s_k; g.out_scale[2] = p.s_v;
    g.out_zero[0] = p.z_q; g.out_zero[1] = p.z_k; g.out_zero[2] = p.z_v;
    g.out = qkv_c; g.ldo = L.ld_qkv;
    if (d.rope) {                       // Q and K ranges rotated ahead of their quantizers, V left alone
      g.rope_cos_sin = p.rope_cos_sin; g.rope_period = S; g.rope_dim = dh; g.rope_groups = 2;
    }
    REPQ_TRY(repq_qgemm(&g, gws, L.gemm_ws, stream));
  }
  REPQ_MARK();
  if (!d.staged_attention) {
    // scores, Softmax codes and P.V in one kernel; it takes the time slot of the scores stage, the two
    // following stages are empty
    repq_attention_desc a{};
    a.batch_outer = d.batch; a.batch_inner = H; a.Lq = S; a.Lk = S; a.d_h = dh; a.bits_qkv = ab;
    a.q_codes = qkv_c; a.ldq_bytes = L.ld_qkv; a.q_stride_outer = int64_t(S) * L.ld_qkv; a.q_stride_inner = head_bytes;
    a.s_q = p.s_q; a.z_q = p.z_q;
    a.k_codes = qkv_c + code_row_bytes(D, ab); a.ldk_bytes = L.ld_qkv; a.k_stride_outer = a.q_stride_outer; a.k_stride_inner = head_bytes;
    a.s_k = p.s_k; a.z_k = p.z_k;
    a.v_codes = qkv_c + 2 * code_row_bytes(D, ab); a.ldv_bytes = L.ld_qkv; a.v_stride_outer = a.q_stride_outer; a.v_stride_inner = head_bytes;
    a.s_v = p.s_v; a.z_v = p.z_v;
    a.alpha = 1.f / sqrtf(float(dh)); a.causal = d.causal; a.bits_p = d.bits_p; a.s_p = p.softmax_s;
    a.out_kind = REPQ_OUT_CODES; a.out_bits = ab; a.out_scale = p.s_attn; a.out_zero = p.z_attn;
    a.out = attn_c; a.ldo = L.ld_a; a.o_stride_outer = int64_t(S) * L.ld_a; a.o_stride_inner = head_bytes;
    a.out_row_sum = asum_attn;
    REPQ_TRY(repq_attention(&a, stream));
    REPQ_MARK();
    REPQ_MARK();
    REPQ_MARK();
  } else {
  {
    // scores = Q K^T / sqrt(d_h) per (batch, head): both operands are activation codes
    repq_gemm_desc g{};
    g.M = S; g.N = S; g.K = dh; g.batch_outer = d.batch; g.batch_inner = H;
    g.a_codes = qkv_c; g.bits_a = ab; g.lda_bytes = L.ld_qkv;
    g.a_stride_outer = int64_t(S) * L.ld_qkv; g.a_stride_inner = head_bytes;
    g.s_a = p.s_q; g.z_a = p.z_q;
    g.w_codes = qkv_c + code_row_bytes(D, ab); g.bits_w = ab; g.ldw_bytes = L.ld_qkv;
    g.w_stride_outer = g.a_stride_outer; g.w_stride_inner = head_bytes;
    g.s_w_scalar = p.s_k; g.z_w_scalar = p.z_k;
    g.alpha = 1.f / sqrtf(float(dh));
    g.causal = d.causal;
    g.out_kind = REPQ_OUT_F32; g.out_groups = 1; g.out_scale[0] = 1.f;
    g.out = scores; g.ldo = L.ld_s;
    g.o_stride_outer = int64_t(H) * S * L.ld_s; g.o_stride_inner = int64_t(S) * L.ld_s;
    REPQ_TRY(repq_qgemm(&g, nullptr, 0, stream));
  }
  REPQ_MARK();
  REPQ_TRY(repq_softmax_log2(scores, REPQ_F32, int64_t(d.batch) * H * S, S, L.ld_s, 1.f, d.causal ? S : 0, 0,
                             p.softmax_s, d.bits_p, p_c, L.ld_p, stream));
  REPQ_MARK();
  {
    repq_pv_desc v{};
    v.batch_outer = d.batch; v.batch_inner = H; v.Lq = S; v.Lk = S; v.d_h = dh;
    v.p_codes = p_c; v.bits_p = d.bits_p; v.ldp_bytes = L.ld_p; v.p_stride_pair = int64_t(S) * L.ld_p;
    v.s_p = p.softmax_s;
    v.v_codes = qkv_c + 2 * code_row_bytes(D, ab); v.bits_v = ab; v.ldv_bytes = L.ld_qkv;
    v.v_stride_outer = int64_t(S) * L.ld_qkv; v.v_stride_inner = head_bytes;
    v.s_v = p.s_v; v.z_v = p.z_v; v.causal = d.causal;
    v.out_kind = REPQ_OUT_CODES; v.out_bits = ab; v.out_scale = p.s_attn; v.out_zero = p.z_attn;
    v.out = attn_c; v.ldo = L.ld_a; v.o_stride_outer = int64_t(S) * L.ld_a; v.o_stride_inner = head_bytes;
    v.out_row_sum = asum_attn;
    REPQ_TRY(repq_pv(&v, stream));
  }
  REPQ_MARK();
  }
  {
    repq_gemm_desc g = linear_desc(d, M, D, D, attn_c, L.ld_a, p.s_attn, p.z_attn, asum_attn, p.proj);
    g.residual = x; g.residual_dtype = d.act_dtype; g.ld_residual = D;
    g.out_kind = d.act_dtype == REPQ_F32 ? REPQ_OUT_F32 : REPQ_OUT_BF16;
    g.out = xbar; g.ldo = D;
    REPQ_TRY(repq_qgemm(&g, gws, L.gemm_ws, stream));
  }
  REPQ_MARK();
  // ---- Y = MLP(LN(X_bar)) + X_bar
  REPQ_TRY(repq_ln_quant(xbar, d.act_dtype, M, D, D, p.ln2_gamma_t, p.ln2_beta_t, d.eps, d.norm_kind, p.ln2_s, p.ln2_z,
                         ab, ln_c, L.ld_a, asum, stream));
  REPQ_MARK();
  {
    const bool swiglu = d.mlp_kind == REPQ_MLP_SWIGLU;
    repq_gemm_desc g = linear_desc(d, M, swiglu ? 2 * d.mlp : d.mlp, D, ln_c, L.ld_a, p.ln2_s, p.ln2_z, asum, p.fc1);
    g.gelu = !swiglu;
    g.glu = swiglu;                     // weight rows (2i, 2i+1) = (gate_i, up_i): d.mlp codes per row leave
    g.out_kind = REPQ_OUT_CODES; g.out_bits = ab; g.out_groups = 1;
    g.out_scale[0] = p.s_hidden; g.out_zero[0] = p.z_hidden;
    g.out = hid_c; g.ldo = L.ld_h; g.out_row_sum = asum_h;
    REPQ_TRY(repq_qgemm(&g, gws, L.gemm_ws, stream));
  }
  REPQ_MARK();
  {
    repq_gemm_desc g = linear_desc(d, M, D, d.mlp, hid_c, L.ld_h, p.s_hidden, p.z_hidden, asum_h, p.fc2);
    g.residual = xbar; g.residual_dtype = d.act_dtype; g.ld_residual = D;
    g.out_kind = d.out_dtype == REPQ_F32 ? REPQ_OUT_F32 : REPQ_OUT_BF16;
    g.out = y; g.ldo = D;
    REPQ_TRY(repq_qgemm(&g, gws, L.gemm_ws, stream));
  }
  REPQ_MARK();
  return REPQ_OK;
}
#undef REPQ_MARK

extern "C" repq_status repq_block_forward(const repq_block_desc* d, const repq_block_params* p, const void* x,
                                          void* y, void* workspace, size_t workspace_bytes, void* stream) {
  return block_forward_impl(d, p, x, y, workspace, workspace_bytes, stream, nullptr);
}

extern "C" repq_status repq_block_forward_timed(const repq_block_desc* d, const repq_block_params* p,
                                                const void* x, void* y, void* workspace, size_t workspace_bytes,
                                                void* stream, float* stage_ms) {
  REPQ_REQUIRE(stage_ms, REPQ_INVALID_ARG, "block_forward_timed: NULL stage_ms");
  cudaEvent_t ev[REPQ_BLOCK_STAGES + 1];
  int made = 0;
  repq_status rc = REPQ_OK;
  for (; made <= REPQ_BLOCK_STAGES; ++made)
    if (cudaEventCreate(&ev[made]) != cudaSuccess) { rc = fail(REPQ_CUDA_ERROR, "cudaEventCreate failed"); break; }
  if (rc == REPQ_OK) rc = block_forward_impl(d, p, x, y, workspace, workspace_bytes, stream, ev);
  if (rc == REPQ_OK && cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess)
    rc = fail(REPQ_CUDA_ERROR, "cudaStreamSynchronize failed: %s", cudaGetErrorString(cudaGetLastError()));
  if (rc == REPQ_OK)
    for (int i = 0; i < REPQ_BLOCK_STAGES; ++i)
      if (cudaEventElapsedTime(&stage_ms[i], ev[i], ev[i + 1]) != cudaSuccess) { rc = fail(REPQ_CUDA_ERROR, "cudaEventElapsedTime failed"); break; }
  for (int i = 0; i < made; ++i) cudaEventDestroy(ev[i]);
  return rc;
}

// ---- allocation-free variant: the workspace is a scratch array inside the library image ------------
//
// `g_static_ws` is device memory that exists on every GPU that loads this library.  On the host its
// name is only a handle for the runtime: the usable device address comes from cudaGetSymbolAddress,
// looked up once per device (with that device current) and cached below.
static __device__ __align__(256) unsigned char g_static_ws[REPQ_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// one slot per device; concurrent first calls may both look the address up, and store the same value
std::atomic<void*> g_static_ws_addr[kMaxDevices];

repq_status static_workspace(void** out) {
  int dev = -1;
  REPQ_CUDA(cudaGetDevice(&dev));
  REPQ_REQUIRE(dev >= 0 && dev < kMaxDevices, REPQ_UNSUPPORTED, "block_forward_static: device index %d not supported", dev);
  void* ptr = g_static_ws_addr[dev].load(std::memory_order_acquire);
  if (ptr == nullptr) {
    REPQ_CUDA(cudaGetSymbolAddress(&ptr, g_static_ws));
    REPQ_REQUIRE(ptr != nullptr, REPQ_CUDA_ERROR, "block_forward_static: scratch array has no device address");
    g_static_ws_addr[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return REPQ_OK;
}
}  // namespace

extern "C" repq_status repq_block_forward_static(const repq_block_desc* d, const repq_block_params* p,
                                                 const void* x, void* y, void* stream) {
  REPQ_REQUIRE(d && p && x && y, REPQ_INVALID_ARG, "block_forward_static: NULL argument");
  REPQ_TRY(validate(*d));
  const size_t need = layout(*d).total;
  REPQ_REQUIRE(need <= size_t(REPQ_STATIC_WORKSPACE_BYTES), REPQ_WORKSPACE_TOO_SMALL,
               "block_forward_static: this block needs %zu bytes of workspace, the built-in scratch holds %zu; "
               "use repq_block_forward with a caller-provided workspace",
               need, size_t(REPQ_STATIC_WORKSPACE_BYTES));
  void* ws = nullptr;
  REPQ_TRY(static_workspace(&ws));
  // The stages overwrite every intermediate they read, and the two row-sum accumulators that must
  // start at zero are cleared inside the stage sequence, so stale contents of earlier calls are harmless.
  return block_forward_impl(d, p, x, y, ws, size_t(REPQ_STATIC_WORKSPACE_BYTES), stream, nullptr);
}

extern "C" repq_status repq_bounded_wait_selftest(int64_t limit_cycles, void* stream) {
  REPQ_REQUIRE(limit_cycles > 0 && limit_cycles <= 2000000000LL, REPQ_INVALID_ARG,
               "bounded_wait_selftest: limit must be between 1 and 2e9 cycles");
  return launch_wait_selftest(limit_cycles, static_cast<cudaStream_t>(stream));
}

extern "C" repq_status repq_device_status(int32_t* status, int reset) {
  REPQ_REQUIRE(status, REPQ_INVALID_ARG, "device_status: NULL argument");
  int32_t* word = device_status_word();
  if (word == nullptr) {            // no kernel with bounded waits has run on this device yet
    *status = 0;
    return REPQ_OK;
  }
  REPQ_CUDA(cudaDeviceSynchronize());
  REPQ_CUDA(cudaMemcpy(status, word, sizeof(int32_t), cudaMemcpyDeviceToHost));
  if (reset) REPQ_CUDA(cudaMemset(word, 0, sizeof(int32_t)));
  REPQ_REQUIRE(*status == 0, REPQ_TIMEOUT, "a bounded device-side wait ran out (code %d): results of that launch are invalid", int(*status));
  return REPQ_OK;
}
