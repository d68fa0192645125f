// Entry points that launch nothing: version, error text, workspace sizing.
#include "ngc_common.cuh"
#include "ngc_plan.h"

namespace ngc {
thread_local int g_last_cuda_error = 0;
}

extern "C" {

int ngc_version(void) { return 100; }

const char* ngc_strerror(int status) {
  switch (status) {
    case NGC_OK: return "ok";
    case NGC_ERR_INVALID_ARG: return "invalid argument";
    case NGC_ERR_UNSUPPORTED: return "shape or dtype not supported by this build";
    case NGC_ERR_WORKSPACE: return "workspace missing or too small";
    case NGC_ERR_CUDA: return "CUDA call failed (see ngc_last_cuda_error)";
    case NGC_ERR_STATIC_SCRATCH:
      return "launch needs more scratch than NGC_STATIC_SCRATCH_BYTES: use the workspace variant or a narrower layer range";
    default: return "unknown status";
  }
}

int ngc_last_cuda_error(void) { return ngc::g_last_cuda_error; }

int ngc_decode_splits(const ngc_cache* c, int layers) {
  if (!ngc::valid_cache(c) || layers <= 0) return 0;
  return ngc::decode_n_split(c, layers);
}

size_t ngc_workspace_bytes(int op, const ngc_cache* c, int G, int n_max, int k_max) {
  switch (op) {
    case NGC_OP_SCORE: return c ? ngc::score_workspace_bytes(c, G, n_max) : 0;
    case NGC_OP_SAMPLE: return c ? ngc::sample_workspace_bytes(c->B, G, n_max) : 0;
    case NGC_OP_LOGPROB: return 0;
    case NGC_OP_COMPACT: return 0;
    case NGC_OP_DECODE: return c ? ngc::decode_workspace_bytes(c, c->L) : 0;
    case NGC_OP_SCORE_BACKWARD: return c ? ngc::score_backward_workspace_bytes(c) : 0;
    default: return 0;
  }
}

}  // extern "C"
