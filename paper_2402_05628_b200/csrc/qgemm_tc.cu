// Placeholder until the tensor-memory GEMM lands: every problem goes to the warp-MMA kernel.
#include "kernels.h"
namespace repq {
bool qgemm_tc_supported(const repq_gemm_desc&) { return false; }
size_t qgemm_tc_workspace(const repq_gemm_desc&) { return 0; }
repq_status qgemm_tc(const repq_gemm_desc&, const EpilogueParams&, void*, size_t, cudaStream_t) {
  return fail(REPQ_UNSUPPORTED, "tensor-memory GEMM not built");
}
int32_t* device_status_word() { return nullptr; }
}  // namespace repq
