// Host-buffer form of the block: a sequence of independent batches whose inputs and outputs live in host
// memory.  The copies and the block's kernels of neighbouring batches overlap: while batch i is computed,
// batch i + 1 is copied in and batch i - 1 is copied out, through two device staging buffers per direction
// and two helper streams.  (Plumbing around the block; the block itself is repq_block_forward.)
#include <mutex>

#include "kernels.h"

namespace repq {
namespace {

constexpr int kMaxDevices = 64;
constexpr int kSlots = 2;

struct Pipeline {                 // per device, created on first use, kept for the life of the process
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr;
  cudaEvent_t copied_in[kSlots] = {}, computed[kSlots] = {}, copied_out[kSlots] = {};
};
Pipeline g_pipe[kMaxDevices];
std::mutex g_pipe_mutex;

repq_status pipeline(Pipeline** out) {
  int dev = -1;
  REPQ_CUDA(cudaGetDevice(&dev));
  REPQ_REQUIRE(dev >= 0 && dev < kMaxDevices, REPQ_UNSUPPORTED, "block_forward_host: device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  Pipeline& P = g_pipe[dev];
  if (!P.ready) {
    REPQ_CUDA(cudaStreamCreateWithFlags(&P.in, cudaStreamNonBlocking));
    REPQ_CUDA(cudaStreamCreateWithFlags(&P.out, cudaStreamNonBlocking));
    REPQ_CUDA(cudaEventCreateWithFlags(&P.start, cudaEventDisableTiming));
    for (int s = 0; s < kSlots; ++s) {
      REPQ_CUDA(cudaEventCreateWithFlags(&P.copied_in[s], cudaEventDisableTiming));
      REPQ_CUDA(cudaEventCreateWithFlags(&P.computed[s], cudaEventDisableTiming));
      REPQ_CUDA(cudaEventCreateWithFlags(&P.copied_out[s], cudaEventDisableTiming));
    }
    P.ready = true;
  }
  *out = &P;
  return REPQ_OK;
}

size_t dtype_size(int dtype) { return dtype == REPQ_F32 ? 4 : 2; }

}  // namespace
}  // namespace repq

using namespace repq;

extern "C" repq_status repq_block_forward_host(const repq_block_desc* d, const repq_block_params* p,
                                               const void* const* x_host, void* const* y_host, int n_batches,
                                               const repq_host_staging* s, void* stream) {
  REPQ_REQUIRE(d && p && x_host && y_host && s, REPQ_INVALID_ARG, "block_forward_host: NULL argument");
  REPQ_REQUIRE(n_batches >= 0, REPQ_INVALID_ARG, "block_forward_host: negative number of batches");
  REPQ_REQUIRE(d->act_dtype == REPQ_F32 || d->act_dtype == REPQ_BF16, REPQ_INVALID_ARG, "block_forward_host: bad act_dtype");
  REPQ_REQUIRE(d->out_dtype == REPQ_F32 || d->out_dtype == REPQ_BF16, REPQ_INVALID_ARG, "block_forward_host: bad out_dtype");
  if (n_batches == 0) return REPQ_OK;
  for (int k = 0; k < kSlots; ++k)
    REPQ_REQUIRE(s->x_dev[k] && s->y_dev[k], REPQ_INVALID_ARG, "block_forward_host: NULL staging buffer");
  REPQ_REQUIRE(s->x_dev[0] != s->x_dev[1] && s->y_dev[0] != s->y_dev[1], REPQ_INVALID_ARG,
               "block_forward_host: the two staging buffers of a direction must differ");
  for (int i = 0; i < n_batches; ++i)
    REPQ_REQUIRE(x_host[i] && y_host[i], REPQ_INVALID_ARG, "block_forward_host: NULL host buffer of batch %d", i);
  const size_t elems = size_t(d->batch) * size_t(d->seq) * size_t(d->dim);
  const size_t x_bytes = elems * dtype_size(d->act_dtype), y_bytes = elems * dtype_size(d->out_dtype);
  Pipeline* P = nullptr;
  REPQ_TRY(pipeline(&P));
  cudaStream_t main = static_cast<cudaStream_t>(stream);

  // the helper streams start after everything already queued on the caller's stream
  REPQ_CUDA(cudaEventRecord(P->start, main));
  REPQ_CUDA(cudaStreamWaitEvent(P->in, P->start, 0));
  REPQ_CUDA(cudaStreamWaitEvent(P->out, P->start, 0));
  for (int i = 0; i < n_batches; ++i) {
    const int k = i % kSlots;
    // copy in: x_dev[k] was last read by the block of batch i - 2
    if (i >= kSlots) REPQ_CUDA(cudaStreamWaitEvent(P->in, P->computed[k], 0));
    REPQ_CUDA(cudaMemcpyAsync(s->x_dev[k], x_host[i], x_bytes, cudaMemcpyHostToDevice, P->in));
    REPQ_CUDA(cudaEventRecord(P->copied_in[k], P->in));
    // block: y_dev[k] was last read by the copy-out of batch i - 2
    REPQ_CUDA(cudaStreamWaitEvent(main, P->copied_in[k], 0));
    if (i >= kSlots) REPQ_CUDA(cudaStreamWaitEvent(main, P->copied_out[k], 0));
    REPQ_TRY(repq_block_forward(d, p, s->x_dev[k], s->y_dev[k], s->workspace, s->workspace_bytes, stream));
    REPQ_CUDA(cudaEventRecord(P->computed[k], main));
    // copy out
    REPQ_CUDA(cudaStreamWaitEvent(P->out, P->computed[k], 0));
    REPQ_CUDA(cudaMemcpyAsync(y_host[i], s->y_dev[k], y_bytes, cudaMemcpyDeviceToHost, P->out));
    REPQ_CUDA(cudaEventRecord(P->copied_out[k], P->out));
  }
  // the caller's stream completes only after the last copies out (and hence after every copy in)
  for (int i = n_batches > kSlots ? n_batches - kSlots : 0; i < n_batches; ++i)
    REPQ_CUDA(cudaStreamWaitEvent(main, P->copied_out[i % kSlots], 0));
  return REPQ_OK;
}
