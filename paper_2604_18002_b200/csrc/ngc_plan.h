// Host-side launch planning shared by the workspace query and the launchers,
// so that both always agree on scratch sizes.
#pragma once

#include <stddef.h>

#include "ngc.h"

namespace ngc {

// Largest candidate count the shared-memory sorter of ngc_sample_evict holds;
// longer lists are sorted in the caller's workspace.
constexpr int kSampleSmemMaxUnits = 16384;

// Number of token-range splits a decode launch over `layers` layers uses.
int decode_n_split(const ngc_cache* c, int layers);
size_t decode_call_scratch_bytes(const ngc_cache* c, int n_layers, size_t* ml_offset);
size_t decode_workspace_bytes(const ngc_cache* c, int layers);

size_t sample_workspace_bytes(int B, int G, int n_max);

size_t score_workspace_bytes(const ngc_cache* c, int G, int n_max);
size_t score_backward_workspace_bytes(const ngc_cache* c);

}  // namespace ngc
