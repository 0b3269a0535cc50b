// Temporary: entry points not implemented yet.
#include "common.h"
using namespace repq;
extern "C" repq_status repq_pv(const repq_pv_desc*, void*) { return fail(REPQ_UNSUPPORTED, "not built yet"); }
extern "C" repq_status repq_block_workspace_bytes(const repq_block_desc*, size_t*) { return fail(REPQ_UNSUPPORTED, "not built yet"); }
extern "C" repq_status repq_block_forward(const repq_block_desc*, const repq_block_params*, const void*, void*, void*, size_t, void*) { return fail(REPQ_UNSUPPORTED, "not built yet"); }
extern "C" repq_status repq_device_status(int32_t* s, int) { if (s) *s = 0; return REPQ_OK; }
