// Host-side helpers shared between translation units of the library (not part of the public ABI).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include "smartgen.h"

namespace sg {
size_t score_workspace_bytes(const sg_shape* shape);
size_t decode_workspace_bytes(const sg_shape* shape, int32_t total_sel, int32_t total_loc);
// Cluster size (CTAs per sequence and KV head) the decode kernel uses for a call of this size.
void decode_plan(const sg_shape* shape, int32_t total_sel, int32_t total_loc, int* csize, int* warps);
}  // namespace sg
