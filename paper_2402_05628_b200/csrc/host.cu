// Host-side entry points: error text, Eq. 6 quantizer parameters, the LayerNorm scale
// reparameterization (Eqs. 10-14) and channel-wise weight quantization (Eqs. 4-6).
// One-time preparation; all arithmetic in float64, results stored as float32 / int32.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <vector>

#include "common.h"

namespace repq {

std::string& last_error_ref() {
  thread_local std::string msg;
  return msg;
}

uint64_t launches();

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

static std::atomic<uint64_t> g_launches{0};
void note_launch(int n) { g_launches.fetch_add(uint64_t(n), std::memory_order_relaxed); }
uint64_t launches() { return g_launches.load(std::memory_order_relaxed); }

}  // namespace repq

using namespace repq;

extern "C" uint64_t repq_launch_count(void) { return repq::launches(); }

extern "C" size_t repq_last_error(char* buf, size_t n) {
  const std::string& m = last_error_ref();
  if (buf && n) {
    size_t k = std::min(n - 1, m.size());
    memcpy(buf, m.data(), k);
    buf[k] = 0;
  }
  return m.size();
}

extern "C" int repq_abi_version(void) { return 5; }

extern "C" repq_status repq_rope_table(int seq, int d_h, double base, float* table) {
  REPQ_REQUIRE(seq > 0 && d_h > 0 && d_h % 2 == 0 && base > 0.0 && table, REPQ_INVALID_ARG, "rope_table: bad argument");
  const int half = d_h / 2;
  for (int i = 0; i < half; ++i) {
    const double theta = std::pow(base, -2.0 * double(i) / double(d_h));
    for (int m = 0; m < seq; ++m) {
      const double ang = double(m) * theta;
      table[(size_t(m) * half + i) * 2 + 0] = float(std::cos(ang));
      table[(size_t(m) * half + i) * 2 + 1] = float(std::sin(ang));
    }
  }
  return REPQ_OK;
}

extern "C" repq_status repq_scale_zero_from_bounds(int n, const float* x_low, const float* x_up,
                                                   int bits, float* s, int32_t* z) {
  REPQ_REQUIRE(n > 0 && x_low && x_up && s && z, REPQ_INVALID_ARG, "scale_zero_from_bounds: bad argument");
  REPQ_REQUIRE(bits_ok(bits), REPQ_INVALID_ARG, "scale_zero_from_bounds: bits must be 4, 6 or 8");
  const double qmax = double(code_max(bits));
  for (int i = 0; i < n; ++i) {
    REPQ_REQUIRE(x_up[i] > x_low[i], REPQ_INVALID_ARG, "scale_zero_from_bounds: x_up <= x_low at %d", i);
    const float sf = float((double(x_up[i]) - double(x_low[i])) / qmax);
    REPQ_REQUIRE(sf > 0.f && std::isfinite(sf), REPQ_INVALID_ARG, "scale_zero_from_bounds: degenerate scale at %d", i);
    s[i] = sf;
    z[i] = int32_t(std::nearbyint(-double(x_low[i]) / double(sf)));
  }
  return REPQ_OK;
}

extern "C" repq_status repq_fold_ln(int D, int N, const float* gamma, const float* beta, const float* s,
                                    const int32_t* z, const float* W, const float* b, float* gamma_t,
                                    float* beta_t, float* s_t, int32_t* z_t, float* W_t, float* b_t) {
  REPQ_REQUIRE(D > 0 && N > 0, REPQ_INVALID_ARG, "fold_ln: D and N must be positive");
  REPQ_REQUIRE(gamma && beta && s && z && W && gamma_t && beta_t && s_t && z_t && W_t && b_t,
               REPQ_INVALID_ARG, "fold_ln: NULL argument");
  double s_sum = 0.0, z_sum = 0.0;
  for (int c = 0; c < D; ++c) {
    REPQ_REQUIRE(s[c] > 0.f && std::isfinite(s[c]), REPQ_INVALID_ARG, "fold_ln: s[%d] is not a positive finite scale", c);
    s_sum += double(s[c]);
    z_sum += double(z[c]);
  }
  const double s_mean = s_sum / D;                                  // s~ = E[s]
  const int32_t z_mean = int32_t(std::nearbyint(z_sum / D));        // z~ = E[z], kept integral
  std::vector<double> r1(D), shift(D);
  for (int c = 0; c < D; ++c) {
    r1[c] = double(s[c]) / s_mean;                                  // r1 = s / s~
    const double r2 = double(z[c] - z_mean);                        // r2 = z - z~
    shift[c] = double(s[c]) * r2;                                   // s * r2
    gamma_t[c] = float(double(gamma[c]) / r1[c]);                   // Eq. 12
    beta_t[c] = float((double(beta[c]) + shift[c]) / r1[c]);
  }
  for (int j = 0; j < N; ++j) {
    const float* wr = W + size_t(j) * D;
    float* wo = W_t + size_t(j) * D;
    double acc = 0.0;
    for (int c = 0; c < D; ++c) {
      const double w = double(wr[c]);
      acc += shift[c] * w;
      wo[c] = float(r1[c] * w);                                     // Eq. 14, weights
    }
    b_t[j] = float((b ? double(b[j]) : 0.0) - acc);                 // Eq. 14, bias
  }
  *s_t = float(s_mean);
  *z_t = z_mean;
  return REPQ_OK;
}

extern "C" repq_status repq_pack_weights(int N, int K, int bits_w, const float* W, uint8_t* codes,
                                         int64_t ld_codes_bytes, float* s_w, int32_t* z_w,
                                         int32_t* w_row_sum) {
  REPQ_REQUIRE(N > 0 && K > 0 && W && codes && s_w && z_w && w_row_sum, REPQ_INVALID_ARG, "pack_weights: bad argument");
  REPQ_REQUIRE(bits_w_ok(bits_w), REPQ_INVALID_ARG, "pack_weights: bits must be 4, 6 or 8 (| REPQ_BYTE_CODES) or 6 | REPQ_PACKED6");
  REPQ_REQUIRE(ld_codes_bytes >= code_row_bytes(K, bits_w) && ld_codes_bytes % 16 == 0, REPQ_ALIGNMENT,
               "pack_weights: ld_codes_bytes must cover a row and be a multiple of 16");
  const int qmax = code_max(bits_w);
  std::vector<int32_t> row(K);
  for (int j = 0; j < N; ++j) {
    const float* wr = W + size_t(j) * K;
    double lo = 0.0, hi = 0.0;
    for (int c = 0; c < K; ++c) {
      REPQ_REQUIRE(std::isfinite(wr[c]), REPQ_INVALID_ARG, "pack_weights: non-finite weight at (%d, %d)", j, c);
      lo = std::min(lo, double(wr[c]));
      hi = std::max(hi, double(wr[c]));
    }
    const double range = hi - lo;
    const float sf = range > 0.0 ? float(range / double(qmax)) : 1.0f;
    const double sd = double(sf);
    const int32_t zj = int32_t(std::nearbyint(-lo / sd));
    int32_t sum = 0;
    for (int c = 0; c < K; ++c) {
      double q = std::nearbyint(double(wr[c]) / sd) + double(zj);
      q = std::min(std::max(q, 0.0), double(qmax));
      row[c] = int32_t(q);
      sum += row[c];
    }
    uint8_t* out = codes + size_t(j) * ld_codes_bytes;
    memset(out, 0, size_t(ld_codes_bytes));
    if (packed4(bits_w)) {
      for (int c = 0; c < K; ++c) out[c >> 1] |= uint8_t(row[c] << ((c & 1) * 4));
    } else if (packed6(bits_w)) {
      for (int c = 0; c < K; ++c) {                 // code c in bits [6c, 6c + 6) of the row
        const int bit = 6 * c;
        const uint32_t v = uint32_t(row[c]) << (bit & 7);
        out[bit >> 3] |= uint8_t(v);
        if ((bit & 7) > 2) out[(bit >> 3) + 1] |= uint8_t(v >> 8);
      }
    } else {
      for (int c = 0; c < K; ++c) out[c] = uint8_t(row[c]);
    }
    s_w[j] = sf;
    z_w[j] = zj;
    w_row_sum[j] = sum;
  }
  return REPQ_OK;
}
