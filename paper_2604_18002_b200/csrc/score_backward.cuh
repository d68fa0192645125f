// Parameter block and the per-token / per-row helpers shared by the kernels of ngc_score_evict_backward
// (paper Section 4.2 scores, differentiated for the loss of Section 4.4).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ngc_common.cuh"
#include "ptx.cuh"

namespace ngc {

constexpr int kBwdMaxRows = 40;                   // (head of the group, window query) rows per strip

struct BwdParams {
  const void* k;
  const void* q_recent;
  const int64_t* seq_off;
  const int32_t* lens;
  const float* logits;         // forward output (log variant only)
  const float* grad_logits;    // [B][G][n_max]
  float4* stats;               // [strips][n_split][kBwdMaxRows] (max, sum e, sum e*P, -)
  float* dq_part;              // [strips][n_split][kBwdMaxRows][128]
  float* grad_q;               // [L][B][Hq][w][128]
  void* grad_k;                // [L][Hkv][R][128] bf16
  int32_t* dev_status;
  int64_t rows_R;
  int L, B, Hq, Hkv, g, w, n_rows, block, lists, G, n_max, log_transform, n_split, lens_lists;
  float scale_log2, inv_sqrt_d;
};

// (m, s, n) <- merge of two partial (max, sum 2^(z-max), sum 2^(z-max) P) triples
__device__ __forceinline__ void merge3(float& m, float& s, float& n, float mo, float so, float no) {
  const float mn = fmaxf(m, mo);
  if (mn == -INFINITY) { s = 0.f; n = 0.f; return; }
  const float fa = ptx::ex2_approx(m - mn), fb = ptx::ex2_approx(mo - mn);
  s = s * fa + so * fb;
  n = n * fa + no * fb;
  m = mn;
}

// dL/dA of a token for the rows of list gi (0 beyond the sequence), in two steps for software pipelining:
// `issue` starts the loads for a token of a LATER tile, `finish`
// turns them into the weight where it is needed.  The empty asm pins the first use of the loaded values to that
// place (otherwise the arithmetic is scheduled right behind the loads and the warp stalls on them at once).
struct TokenWeightRaw { float up, lg, f; };
__device__ __forceinline__ TokenWeightRaw token_weight_issue(const BwdParams& p, int b, int gi, int t, int T_b, float inv_rows) {
  TokenWeightRaw raw = {0.f, 0.f, 0.f};
  if (t < T_b) {
    const int u = p.block == 1 ? t : t / p.block;
    if (u < p.n_max) {
      const int size = p.block == 1 ? 1 : min((u + 1) * p.block, T_b) - u * p.block;
      const int64_t idx = ((int64_t)b * p.G + gi) * p.n_max + u;
      raw.f = inv_rows / (float)size;
      raw.up = p.grad_logits[idx];
      if (p.log_transform) raw.lg = p.logits[idx];
    }
  }
  return raw;
}
__device__ __forceinline__ float token_weight_finish(const BwdParams& p, TokenWeightRaw raw) {
  asm volatile("" : "+f"(raw.up), "+f"(raw.lg));
  float up = raw.up;
  if (p.log_transform) up *= __expf(-raw.lg);                 // d log s = ds / s
  return up * raw.f;
}

// rows of list gi: layers x KV heads feeding it x group size x window queries that exist
__device__ __forceinline__ float inv_list_rows(const BwdParams& p, int T_b) {
  const int w_eff = min(p.w, T_b);
  const int strips = p.lists == NGC_LISTS_SHARED ? p.L * p.Hkv : (p.lists == NGC_LISTS_PER_LAYER ? p.Hkv : 1);
  return 1.f / (float)(strips * p.g * w_eff);
}

// Last visible token of column c of S (row c of the strip = head-in-group c / w, window slot c % w); -1: unused.
__device__ __forceinline__ int column_limit(const BwdParams& p, int c, int T_b) {
  const int jc = c % p.w;
  return (c < p.n_rows && jc >= p.w - min(p.w, T_b)) ? T_b - p.w + jc : -1;
}

// The gradient pass on the 5th-generation tensor cores (score_backward_umma.cu): dK and the per-range dQ partials.
int launch_score_bwd_umma(const BwdParams& p, const void* k, void* grad_k, int64_t rows, int planes, int64_t items, cudaStream_t stream);

}  // namespace ngc
