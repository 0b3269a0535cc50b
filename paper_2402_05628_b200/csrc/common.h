// Shared host-side plumbing of the repq library: error reporting and argument checks.
#pragma once
#include <cuda_runtime.h>
#include <cstdarg>
#include <cstdint>
#include <cstdio>
#include <string>

#include "../../include/repq.h"

namespace repq {

std::string& last_error_ref();

inline repq_status fail(repq_status code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  last_error_ref() = buf;
  return code;
}

#define REPQ_REQUIRE(cond, code, ...) \
  do {                                \
    if (!(cond)) return ::repq::fail((code), __VA_ARGS__); \
  } while (0)

#define REPQ_CUDA(call)                                                                   \
  do {                                                                                    \
    cudaError_t e__ = (call);                                                             \
    if (e__ != cudaSuccess)                                                               \
      return ::repq::fail(REPQ_CUDA_ERROR, "%s failed: %s", #call, cudaGetErrorString(e__)); \
  } while (0)

#define REPQ_TRY(call)                   \
  do {                                   \
    repq_status s__ = (call);            \
    if (s__ != REPQ_OK) return s__;      \
  } while (0)

// A `bits` value = quantizer width (4, 6, 8) | optional REPQ_BYTE_CODES.
inline int quant_bits(int b) { return b & 0xFF; }
inline bool bits_ok(int b) {
  const int q = quant_bits(b);
  return (b & ~(0xFF | REPQ_BYTE_CODES)) == 0 && (q == 4 || q == 6 || q == 8);
}
inline bool packed4(int b) { return b == 4; }                        // two codes per byte
inline bool packed6(int b) { return b == (6 | REPQ_PACKED6); }       // four codes in three bytes (weights only)
inline bool bits_w_ok(int b) { return bits_ok(b) || packed6(b); }
inline int code_max(int b) { return (1 << quant_bits(b)) - 1; }
inline int64_t code_row_bytes(int64_t n, int bits) { return packed4(bits) ? (n + 1) / 2 : packed6(bits) ? (n * 3 + 3) / 4 : n; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

int sm_count();

// Launch accounting (repq_launch_count).
void note_launch(int n = 1);

// Kernels of one stream that follow each other are launched with programmatic stream serialization: the next
// kernel may be scheduled, and run its prologue (barrier setup, tensor-memory allocation, parameter staging), as
// SMs drain from the one before.  Such a kernel calls grid_dependency_wait() before its first access to global
// memory that an earlier kernel may have written or may still read, and grid_dependency_trigger() once it has
// started (both are no-ops in a kernel launched the plain way).
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

}  // namespace repq
