// ngc_score_evict_backward: gradient of the eviction scores (paper Section 4.2) with respect to
// the recent queries and the keys -- the path on which the eviction loss of Section 4.4 reaches
// the model (Section 4.5 recomputes the scores on the autograd graph for exactly this).
//
// With P[t] = grad_logits[unit(t)] / |unit(t)| / n_rows (the same for every attention row r of the
// list; also divided by the unit's score when the logit is log s), A = softmax rows, c[r] = sum_t
// A[r][t] P[t]:
//   dz[r][t] = A[r][t] (P[t] - c[r]) / sqrt(d),   dq[r] = sum_t dz[r][t] k[t],   dk[t] = sum_r dz[r][t] q[r].
//
// bf16, d = 128, at most 40 rows per strip (the shapes of the streaming forward kernel).  Two persistent
// launches on the 5th-generation tensor cores stream K by TMA (score_backward_umma.cu):
//   1. per (strip, token range): row max, sum of exponentials and sum of exponentials times P;
//   2. same geometry: the merged statistics give A and c; S is recomputed, dz formed, dK = dz Q written out as
//      bf16 and dQ += dz^T K accumulated in tensor memory.
// A strip that was cut into several token ranges leaves per-range dQ partials in the workspace, and a third small
// kernel adds them in a fixed order (no float atomics: results are reproducible); an uncut strip writes grad_q itself.
#include <cuda_bf16.h>


#include "kv_map.cuh"
#include "ngc_common.cuh"
#include "ngc_plan.h"
#include "ptx.cuh"
#include "score_backward.cuh"

namespace ngc {
namespace {

constexpr int kTileT = 128;                       // tokens per tile of the streaming kernels
constexpr int kMaxRows = kBwdMaxRows;

// ---------------------------------------------------------------- pass 3: sum the ranges of a strip

__global__ void __launch_bounds__(128) score_bwd_reduce_kernel(BwdParams p) {
  const int strip = blockIdx.x / p.n_rows, r = blockIdx.x % p.n_rows;
  const int h = strip % p.Hkv, b = (strip / p.Hkv) % p.B, l = strip / (p.Hkv * p.B);
  const int hl = r / p.w, j = r - hl * p.w;
  float acc = 0.f;
  for (int s = 0; s < p.n_split; ++s) acc += p.dq_part[(((int64_t)strip * p.n_split + s) * kMaxRows + r) * 128 + threadIdx.x];
  p.grad_q[((((int64_t)l * p.B + b) * p.Hq + h * p.g + hl) * p.w + j) * 128 + threadIdx.x] = acc;
}

constexpr int kTargetCtas = 148 * 4;              // items wanted for an even spread over the persistent CTAs

int bwd_n_split(const ngc_cache* c) {
  const int64_t strips = (int64_t)c->L * c->B * c->Hkv;
  if (strips >= kTargetCtas) return 1;
  int ns = (int)((kTargetCtas + strips - 1) / strips);
  const int by_len = (c->max_len + 4 * kTileT - 1) / (4 * kTileT);
  if (ns > by_len) ns = by_len;
  if (ns > 64) ns = 64;
  return ns < 1 ? 1 : ns;
}

}  // namespace

size_t score_backward_workspace_bytes(const ngc_cache* c) {
  const size_t items = (size_t)c->L * c->B * c->Hkv * bwd_n_split(c);
  return align256(items * kMaxRows * 16) + align256(items * kMaxRows * 128 * 4);
}

}  // namespace ngc

extern "C" int ngc_score_evict_backward(const ngc_cache* c, const void* q_recent, int w, int block, int lists, int log_transform,
                                        const float* logits, const float* grad_logits, int n_max,
                                        float* grad_q_recent, void* grad_k,
                                        void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream_) {
  NGC_API_RANGE("ngc_score_evict_backward");
  using namespace ngc;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!valid_cache(c) || !q_recent || !grad_logits || !grad_q_recent || !grad_k || w <= 0 || w > 16 || block <= 0 || lists < 0 ||
      lists > 2 || n_max <= 0 || (log_transform && !logits))
    return NGC_ERR_INVALID_ARG;
  const int g = c->Hq / c->Hkv;
  if (c->dtype != NGC_BF16 || c->d != 128 || g * w > kMaxRows || c->rows >= 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  if ((((uintptr_t)c->k | (uintptr_t)q_recent | (uintptr_t)grad_k) & 15) != 0) return NGC_ERR_INVALID_ARG;
  if (c->lens_lists != 0 && c->lens_lists != lists) return NGC_ERR_INVALID_ARG;
  if ((int64_t)n_max * block < c->max_len) return NGC_ERR_INVALID_ARG;
  const size_t q_elems = (size_t)c->L * c->B * c->Hq * w * 128;
  if (c->rows == 0 || c->max_len == 0) {
    NGC_CUDA_TRY(cudaMemsetAsync(grad_q_recent, 0, q_elems * 4, stream));
    return NGC_OK;
  }
  const size_t need = score_backward_workspace_bytes(c);
  if (!ws || ws_bytes < need || ((uintptr_t)ws & 255)) return NGC_ERR_WORKSPACE;

  BwdParams p;
  p.k = c->k; p.q_recent = q_recent; p.seq_off = c->seq_off; p.lens = c->lens;
  p.logits = logits; p.grad_logits = grad_logits;
  p.n_split = bwd_n_split(c);
  const size_t items = (size_t)c->L * c->B * c->Hkv * p.n_split;
  p.stats = (float4*)ws;
  p.dq_part = (float*)((char*)ws + align256(items * kMaxRows * 16));
  p.grad_q = grad_q_recent; p.grad_k = grad_k; p.dev_status = dev_status;
  p.rows_R = c->rows;
  p.L = c->L; p.B = c->B; p.Hq = c->Hq; p.Hkv = c->Hkv; p.g = g; p.w = w; p.n_rows = g * w;
  p.block = block; p.lists = lists; p.G = lists_G(lists, c->L, c->Hkv); p.n_max = n_max; p.log_transform = log_transform;
  p.lens_lists = c->lens_lists;
  p.inv_sqrt_d = 1.0f / sqrtf((float)c->d);
  p.scale_log2 = p.inv_sqrt_d * 1.4426950408889634f;
  if (items > 0x7fffffffULL) return NGC_ERR_UNSUPPORTED;
  int rc = launch_score_bwd_umma(p, c->k, grad_k, c->rows, c->L * c->Hkv, (int64_t)items, stream);
  if (rc != NGC_OK) return rc;
  if (p.n_split == 1) return NGC_OK;      // one range per strip: the gradient pass wrote grad_q itself
  score_bwd_reduce_kernel<<<(unsigned)(c->L * c->B * c->Hkv * p.n_rows), 128, 0, stream>>>(p);
  return launch_status();
}
