// Host-side helpers shared between translation units of the library (not part of the public ABI).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include "smartgen.h"

namespace sg {
size_t score_workspace_bytes(const sg_shape* shape);
size_t decode_workspace_bytes(const sg_shape* shape, int32_t total_sel, int32_t total_loc);
// Tokens per split-KV work item chosen for a decode call of this size (a multiple of 64).
int decode_chunk_tokens(const sg_shape* shape, int32_t total_sel, int32_t total_loc);
// Cluster size of the fused decode mode for this call, or 0 when the two-kernel mode is used.
int decode_cluster_size(const sg_shape* shape, int32_t total_sel, int32_t total_loc);
}  // namespace sg
