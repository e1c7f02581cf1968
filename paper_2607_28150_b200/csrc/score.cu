#include "common.cuh"
#include "launch.h"
namespace sg { size_t score_workspace_bytes(const sg_shape*) { return 0; } }
extern "C" sg_status sg_score(const sg_shape*, const void*, const void*, float*, void*, size_t, int32_t*, void*) {
  return SG_ERR_UNSUPPORTED;
}
