// Per-channel dual clipping (Sec. III-D, Eqs. 18-20): the step that hands the channel-wise quantizer of the
// LayerNorm activations its bounds, just before the scale reparameterization.  Every channel d learns two factors,
//     x_up = max_d * sigmoid(alpha1_d),   x_low = min_d * sigmoid(alpha2_d)                      (Eqs. 18-19)
// by Adam on ||X'_{:,d} - X^'_{:,d}||^2 (Eq. 20), X^' the de-quantized channel-wise quantization (Eqs. 4-6) on those
// bounds.  The round operations are passed straight through in the backward direction and the clip passes the
// gradient on [0, 2^b - 1] inclusive: with u = x/s, zc = -x_low/s, r = round(u), z = round(zc), q = clip(r + z),
//     inside the clip   dx^/ds = r - u            dx^/dx_low (s fixed) = 0
//     clipped           dx^/ds = q - z + zc       dx^/dx_low (s fixed) = 1
// and s = (x_up - x_low) / (2^b - 1).
//
// Channels are independent, so the whole optimisation of a channel stays inside one CTA: a CTA owns 8 neighbouring
// channels (one 32-byte sector per token row) and 32 token lanes; every iteration is one pass over the CTA's slab of
// the activations (L2-resident for calibration-sized inputs), a shared-memory reduction of three sums per channel,
// and the Adam update by the channel's first thread.  Arithmetic is float64 throughout (the decisions of the two
// round operations steer the gradient).  No scratch memory, no atomics, no inter-CTA traffic.
#include <cuda_bf16.h>

#include <cmath>

#include "common.h"

namespace repq {
namespace {

constexpr int kCh = 8;            // channels per CTA
constexpr int kLanes = 32;        // token lanes per channel
constexpr int kThreads = kCh * kLanes;

struct ClipParams {
  const float* x; int64_t n, ldx; int D;
  double Q; int iters; double lr, alpha0, beta1, beta2, eps;
  float* x_low; float* x_up; double* loss;
};

__device__ __forceinline__ double sigmoid(double a) { return 1.0 / (1.0 + exp(-a)); }

__global__ void __launch_bounds__(kThreads) dual_clip_kernel(ClipParams P) {
  __shared__ double red[3][kLanes][kCh];
  __shared__ double sh_s[kCh], sh_low[kCh];
  const int ch = threadIdx.x % kCh, lane = threadIdx.x / kCh;
  const int d = blockIdx.x * kCh + ch;
  const bool on = d < P.D;
  const float* col = P.x + (on ? d : 0);

  // ---- extremes of the channel
  double mx = -INFINITY, mn = INFINITY;
  if (on)
    for (int64_t t = lane; t < P.n; t += kLanes) {
      const double v = double(__ldg(col + t * P.ldx));
      mx = fmax(mx, v);
      mn = fmin(mn, v);
    }
  red[0][lane][ch] = mx;
  red[1][lane][ch] = mn;
  __syncthreads();
  double x_max = 0.0, x_min = 0.0;
  // state of the channel's first thread
  double a1 = P.alpha0, a2 = P.alpha0, m1 = 0.0, v1 = 0.0, m2 = 0.0, v2 = 0.0, sg1 = 0.0, sg2 = 0.0;
  double b1t = 1.0, b2t = 1.0;
  if (lane == 0) {
    x_max = red[0][0][ch];
    x_min = red[1][0][ch];
    for (int l = 1; l < kLanes; ++l) {
      x_max = fmax(x_max, red[0][l][ch]);
      x_min = fmin(x_min, red[1][l][ch]);
    }
  }
  double loss_first = 0.0;
  for (int it = 0; it <= P.iters; ++it) {
    // the channel's quantizer for this iteration (Eq. 6 on the bounds of Eqs. 18-19)
    if (lane == 0) {
      sg1 = sigmoid(a1);
      sg2 = sigmoid(a2);
      const double up = x_max * sg1, low = x_min * sg2;
      sh_s[ch] = (up - low) / P.Q;
      sh_low[ch] = low;
    }
    __syncthreads();
    const double s = sh_s[ch], low = sh_low[ch];
    const double zc = -low / s, z = rint(zc);
    double acc_loss = 0.0, acc_ds = 0.0, acc_dl = 0.0;
    // a channel whose bounds coincide (a constant channel, or extremes of 0) has no quantizer to learn: its sums stay
    // 0, its factors keep their starting value and the contracted extremes are returned as they are
    if (on && s > 0.0)
      for (int64_t t = lane; t < P.n; t += kLanes) {
        const double x = double(__ldg(col + t * P.ldx));
        const double u = x / s, r = rint(u), pre = r + z;
        const double q = fmin(fmax(pre, 0.0), P.Q);
        const double e = s * (q - z) - x;
        const bool inside = pre >= 0.0 && pre <= P.Q;
        acc_loss += e * e;
        acc_ds += 2.0 * e * (inside ? r - u : q - z + zc);
        acc_dl += inside ? 0.0 : 2.0 * e;
      }
    red[0][lane][ch] = acc_loss;
    red[1][lane][ch] = acc_ds;
    red[2][lane][ch] = acc_dl;
    __syncthreads();
    if (lane == 0) {
      double loss = 0.0, dL_ds = 0.0, dL_dl = 0.0;
      for (int l = 0; l < kLanes; ++l) {
        loss += red[0][l][ch];
        dL_ds += red[1][l][ch];
        dL_dl += red[2][l][ch];
      }
      if (it == 0) loss_first = loss;
      if (it == P.iters) {
        // the pass after the last update: the objective that the returned bounds reach
        if (on) {
          P.x_up[d] = float(x_max * sg1);
          P.x_low[d] = float(x_min * sg2);
          if (P.loss) {
            P.loss[d] = loss_first;
            P.loss[P.D + d] = loss;
          }
        }
      } else {
        const double g1 = dL_ds / P.Q * x_max * sg1 * (1.0 - sg1);
        const double g2 = (dL_dl - dL_ds / P.Q) * x_min * sg2 * (1.0 - sg2);
        m1 = P.beta1 * m1 + (1.0 - P.beta1) * g1;
        v1 = P.beta2 * v1 + (1.0 - P.beta2) * g1 * g1;
        m2 = P.beta1 * m2 + (1.0 - P.beta1) * g2;
        v2 = P.beta2 * v2 + (1.0 - P.beta2) * g2 * g2;
        b1t *= P.beta1;
        b2t *= P.beta2;
        a1 -= P.lr * (m1 / (1.0 - b1t)) / (sqrt(v1 / (1.0 - b2t)) + P.eps);
        a2 -= P.lr * (m2 / (1.0 - b1t)) / (sqrt(v2 / (1.0 - b2t)) + P.eps);
      }
    }
    // the next iteration's writes of sh_s / red follow this barrier
    __syncthreads();
  }
}

// Full-precision normalisation of the calibration batch (Eq. 9; mean-free variant for RMS): the activations the
// clipping factors are learned on.  One CTA per row at a time, mean and centred variance in float32 with a
// float64 block reduction, float32 output.  Calibration-time only: the inference path never forms X'.
template <typename T>
__global__ void __launch_bounds__(256) layernorm_kernel(const T* __restrict__ x, int64_t rows, int D, int64_t ldx,
                                                        const float* __restrict__ gamma, const float* __restrict__ beta,
                                                        float eps, int rms, float* __restrict__ y, int64_t ldy) {
  __shared__ double red[8];
  __shared__ float bc;
  auto block_sum = [&](double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                               // the previous use of red / bc is over
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int i = 0; i < 8; ++i) t += red[i];
      bc = float(t / double(D));
    }
    __syncthreads();
    return bc;
  };
  auto ld = [](const T* p) {
    if constexpr (sizeof(T) == 2) return __bfloat162float(*p);
    else return float(*p);
  };
  for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const T* xr = x + r * ldx;
    double acc = 0.0;
    if (!rms)
      for (int c = threadIdx.x; c < D; c += 256) acc += double(ld(xr + c));
    const float mu = rms ? 0.f : block_sum(acc);
    acc = 0.0;
    for (int c = threadIdx.x; c < D; c += 256) {
      const float dlt = ld(xr + c) - mu;
      acc += double(dlt) * double(dlt);
    }
    const float rstd = rsqrtf(block_sum(acc) + eps);
    for (int c = threadIdx.x; c < D; c += 256)
      y[r * ldy + c] = fmaf((ld(xr + c) - mu) * rstd, __ldg(gamma + c), __ldg(beta + c));
  }
}

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_layernorm(const void* x, int x_dtype, int64_t rows, int D, int64_t ldx, const float* gamma,
                                      const float* beta, float eps, int norm_kind, float* y, int64_t ldy, void* stream) {
  REPQ_REQUIRE(rows >= 0 && D > 0 && ldx >= D && ldy >= D, REPQ_INVALID_ARG, "layernorm: bad sizes");
  if (rows == 0) return REPQ_OK;
  REPQ_REQUIRE(x && gamma && beta && y, REPQ_INVALID_ARG, "layernorm: NULL pointer");
  REPQ_REQUIRE(x_dtype == REPQ_F32 || x_dtype == REPQ_BF16, REPQ_INVALID_ARG, "layernorm: x_dtype must be REPQ_F32 or REPQ_BF16");
  REPQ_REQUIRE(norm_kind == REPQ_NORM_LAYERNORM || norm_kind == REPQ_NORM_RMS, REPQ_INVALID_ARG, "layernorm: unknown norm_kind");
  REPQ_REQUIRE(eps >= 0.f, REPQ_INVALID_ARG, "layernorm: eps must be non-negative");
  const int grid = int(rows < 4096 ? rows : 4096);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rms = norm_kind == REPQ_NORM_RMS;
  if (x_dtype == REPQ_F32)
    layernorm_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(x), rows, D, ldx, gamma, beta, eps, rms, y, ldy);
  else
    layernorm_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), rows, D, ldx, gamma, beta, eps, rms, y, ldy);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}

extern "C" repq_status repq_dual_clip(const float* x, int64_t n, int D, int64_t ldx, int bits, int iters, float lr,
                                      float alpha0, float* x_low, float* x_up, double* loss, void* stream) {
  REPQ_REQUIRE(x && x_low && x_up, REPQ_INVALID_ARG, "dual_clip: NULL pointer");
  REPQ_REQUIRE(n > 0 && D > 0 && ldx >= D, REPQ_INVALID_ARG, "dual_clip: n and D must be positive, ldx >= D");
  REPQ_REQUIRE(bits == 4 || bits == 6 || bits == 8, REPQ_INVALID_ARG, "dual_clip: bits must be 4, 6 or 8");
  REPQ_REQUIRE(iters >= 0 && iters <= 100000 && lr > 0.f, REPQ_INVALID_ARG, "dual_clip: iters must be 0..100000 and lr positive");
  ClipParams P{};
  P.x = x; P.n = n; P.ldx = ldx; P.D = D;
  P.Q = double((1 << bits) - 1);
  P.iters = iters; P.lr = double(lr); P.alpha0 = double(alpha0);
  P.beta1 = 0.9; P.beta2 = 0.999; P.eps = 1e-8;
  P.x_low = x_low; P.x_up = x_up; P.loss = loss;
  const int grid = (D + kCh - 1) / kCh;
  dual_clip_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(P);
  REPQ_CUDA(cudaGetLastError());
  note_launch();
  return REPQ_OK;
}
