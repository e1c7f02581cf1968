// Status strings, the per-thread CUDA error slot and the workspace-size query of the C ABI.
#include "common.cuh"
#include "launch.h"

namespace sg {
thread_local int g_last_cuda_error = 0;
}

extern "C" const char* sg_strerror(sg_status status) {
  switch (status) {
    case SG_OK: return "ok";
    case SG_ERR_INVALID: return "invalid argument (null or misaligned pointer, bad shape, budget above prompt length)";
    case SG_ERR_UNSUPPORTED: return "unsupported shape (head_dim, head grouping or window beyond the built kernels)";
    case SG_ERR_WORKSPACE: return "workspace too small (see sg_workspace_bytes)";
    case SG_ERR_CUDA: return "a CUDA call failed (see sg_last_cuda_error)";
    case SG_ERR_INDEX: return "an index outside its sequence was skipped";
    case SG_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
  }
  return "unknown status";
}

extern "C" int sg_last_cuda_error(void) { return sg::g_last_cuda_error; }

extern "C" size_t sg_workspace_bytes(int op, const sg_shape* shape, int32_t total_sel, int32_t total_loc) {
  if (!shape) return 0;
  switch (op) {
    case SG_OP_SCORE: return sg::score_workspace_bytes(shape);
    case SG_OP_SPARSE_DECODE_ATTN: return sg::decode_workspace_bytes(shape, total_sel, total_loc);
    default: return 0;
  }
}
