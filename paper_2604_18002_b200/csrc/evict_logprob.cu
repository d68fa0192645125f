// ngc_evict_logprob: Eq. (1) of the paper (Section 4.3), fp64.
//
// One CTA per list.  With e_t = exp(s_t - M) (M = largest candidate logit) the
// partition function of step j is the mass still present:
//   rem_j = sum_{t never drawn} e_t + sum_{i >= j} e_sigma_i ,
// so all K of them come from one scan over sigma taken from the tail, by
// additions only (the remaining-mass bookkeeping the paper mentions after
// Eq. (1), arranged so that nothing is subtracted).  Reductions and the scan
// use a fixed tree order: results are reproducible run to run.
//
// Lists of at most 32 units (the paper's own setting: block-level lists of
// 16-22 units, Section 5.1) take a warp each, eight lists per CTA, the whole
// list in registers and every reduction a shuffle.
#include "ngc_common.cuh"

namespace ngc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct LogprobParams {
  const float* logits;
  const int32_t* n;
  const int32_t* n_protect;
  const int32_t* budget;
  const int32_t* kept_order;
  double* logp;
  int32_t* dev_status;
  int G, n_max, k_max;
};

__device__ double block_sum(double v, double* s_red) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) t += s_red[w];
  return t;
}

__global__ void __launch_bounds__(kThreads) logprob_kernel(LogprobParams p) {
  extern __shared__ uint32_t bitmap[];
  __shared__ double s_red[kWarps];
  __shared__ float s_redf[kWarps];
  __shared__ int s_bad;

  const int64_t li = blockIdx.x;
  const int64_t outer = li / p.G;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n[outer];
  const int P = p.n_protect ? p.n_protect[outer] : 0;
  const int K = p.budget[outer];
  const int Kp = K - P;
  const float* s = p.logits + li * p.n_max;
  const int32_t* sigma = p.kept_order + li * p.k_max;
  const double kNaN = __longlong_as_double(0x7ff8000000000000LL);

  if (!(P >= 0 && P <= K && K <= n && n <= p.n_max && Kp <= p.k_max)) {
    if (tid == 0) { set_dev_status(p.dev_status, NGC_DEV_BAD_COUNTS); p.logp[li] = kNaN; }
    return;
  }
  // ---- mark the drawn units; refuse repeats and out-of-range entries ----
  if (tid == 0) s_bad = 0;
  for (int w = tid; w < (n + 31) / 32; w += kThreads) bitmap[w] = 0u;
  __syncthreads();
  int bad = 0;
  for (int j = tid; j < Kp; j += kThreads) {
    const int t = sigma[j];
    if (t < P || t >= n) bad = 1;
    else if (atomicOr(&bitmap[t >> 5], 1u << (t & 31)) & (1u << (t & 31))) bad = 1;
  }
  if (bad) atomicOr(&s_bad, 1);
  __syncthreads();
  if (s_bad) {
    if (tid == 0) { set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT); p.logp[li] = kNaN; }
    return;
  }
  if (Kp == 0) {
    if (tid == 0) p.logp[li] = 0.0;
    return;
  }
  // ---- M = max candidate logit ----
  float mx = -INFINITY;
  int nan_seen = 0;
  for (int t = P + tid; t < n; t += kThreads) {
    const float v = s[t];
    if (v != v) nan_seen = 1;
    mx = fmaxf(mx, v);
  }
  mx = warp_max(mx);
  if (lane == 0) s_redf[warp] = mx;
  if (nan_seen) atomicOr(&s_bad, 1);
  __syncthreads();
  mx = s_redf[0];
#pragma unroll
  for (int w = 1; w < kWarps; ++w) mx = fmaxf(mx, s_redf[w]);
  if (s_bad) {
    if (tid == 0) { set_dev_status(p.dev_status, NGC_DEV_NAN_LOGIT); p.logp[li] = kNaN; }
    return;
  }
  const double M = (double)mx;
  // ---- mass of the candidates that are never drawn ----
  double u = 0.0;
  for (int t = P + tid; t < n; t += kThreads)
    if (!((bitmap[t >> 5] >> (t & 31)) & 1u)) u += exp((double)s[t] - M);
  double carry = block_sum(u, s_red);
  // ---- scan sigma from the tail: rem_j = carry + e_sigma_j + ... ----
  double acc = 0.0;
  for (int base = 0; base < Kp; base += kThreads) {
    const int j = Kp - 1 - (base + tid);
    double sj = 0.0, e = 0.0;
    if (j >= 0) { sj = (double)s[sigma[j]] - M; e = exp(sj); }
    double incl = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    double off = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      if (w < warp) off += s_red[w];
      tot += s_red[w];
    }
    if (j >= 0) acc += sj - log(carry + off + incl);
    carry += tot;
  }
  const double total = block_sum(acc, s_red);
  if (tid == 0) p.logp[li] = total;
}

// ---------------------------------------------------------------- gradient with respect to the logits
//
// d logp / d s_i = [i drawn] - e_i * C(i),  C(i) = sum over the steps j at which i was still a
// candidate of 1 / rem_j: steps 1..m for the unit drawn at step m, all K steps for a unit never
// drawn.  rem_j comes from the same tail scan as the forward value; a second scan, from the
// front, accumulates the reciprocals.

struct GradParams {
  LogprobParams f;
  const double* grad_logp;   // [lists] or null (= 1)
  float* grad_logits;        // [lists][n_max]
};

__global__ void __launch_bounds__(kThreads) logprob_grad_kernel(GradParams g) {
  extern __shared__ __align__(8) unsigned char smem_raw[];
  __shared__ double s_red[kWarps];
  __shared__ float s_redf[kWarps];
  __shared__ int s_bad;
  const LogprobParams& p = g.f;

  const int64_t li = blockIdx.x;
  const int64_t outer = li / p.G;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n[outer];
  const int P = p.n_protect ? p.n_protect[outer] : 0;
  const int K = p.budget[outer];
  const int Kp = K - P;
  const float* s = p.logits + li * p.n_max;
  const int32_t* sigma = p.kept_order + li * p.k_max;
  float* out = g.grad_logits + li * p.n_max;
  double* inv = reinterpret_cast<double*>(smem_raw);                                   // [min(k_max, n_max)]
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(smem_raw + (size_t)min(p.k_max, p.n_max) * 8);
  const float kNaNf = __int_as_float(0x7fc00000);

  int fail = 0;
  if (!(P >= 0 && P <= K && K <= n && n <= p.n_max && Kp <= p.k_max)) fail = NGC_DEV_BAD_COUNTS;
  if (!fail) {
    if (tid == 0) s_bad = 0;
    for (int w = tid; w < (n + 31) / 32; w += kThreads) bitmap[w] = 0u;
    __syncthreads();
    int bad = 0;
    for (int j = tid; j < Kp; j += kThreads) {
      const int t = sigma[j];
      if (t < P || t >= n) bad = 1;
      else if (atomicOr(&bitmap[t >> 5], 1u << (t & 31)) & (1u << (t & 31))) bad = 1;
    }
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    if (s_bad) fail = NGC_DEV_BAD_KEPT;
  }
  float mx = -INFINITY;
  if (!fail) {
    int nan_seen = 0;
    for (int t = P + tid; t < n; t += kThreads) {
      const float v = s[t];
      if (v != v) nan_seen = 1;
      mx = fmaxf(mx, v);
    }
    mx = warp_max(mx);
    if (lane == 0) s_redf[warp] = mx;
    if (nan_seen) atomicOr(&s_bad, 1);
    __syncthreads();
    mx = s_redf[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) mx = fmaxf(mx, s_redf[w]);
    if (s_bad) fail = NGC_DEV_NAN_LOGIT;
  }
  if (fail) {
    if (tid == 0) set_dev_status(p.dev_status, fail);
    for (int t = tid; t < p.n_max; t += kThreads) out[t] = kNaNf;
    return;
  }
  const double up = g.grad_logp ? g.grad_logp[li] : 1.0;
  const double M = (double)mx;
  // ---- mass of the candidates that are never drawn ----
  double u = 0.0;
  for (int t = P + tid; t < n; t += kThreads)
    if (!((bitmap[t >> 5] >> (t & 31)) & 1u)) u += exp((double)s[t] - M);
  double carry = block_sum(u, s_red);
  // ---- tail scan: inv[j] = 1 / rem_j ----
  for (int base = 0; base < Kp; base += kThreads) {
    const int j = Kp - 1 - (base + tid);
    const double e = j >= 0 ? exp((double)s[sigma[j]] - M) : 0.0;
    double incl = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    double off = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      if (w < warp) off += s_red[w];
      tot += s_red[w];
    }
    if (j >= 0) inv[j] = 1.0 / (carry + off + incl);
    carry += tot;
  }
  __syncthreads();
  // ---- front scan: C_j = inv[0] + ... + inv[j]; the unit drawn at step j gets 1 - e * C_j ----
  double c_carry = 0.0;
  for (int base = 0; base < Kp; base += kThreads) {
    const int j = base + tid;
    double incl = j < Kp ? inv[j] : 0.0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    double off = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      if (w < warp) off += s_red[w];
      tot += s_red[w];
    }
    if (j < Kp) {
      const int t = sigma[j];
      out[t] = (float)(up * (1.0 - exp((double)s[t] - M) * (c_carry + off + incl)));
    }
    c_carry += tot;
  }
  // ---- everything else: never drawn -> -e * C_K; protected units and padding -> 0 ----
  for (int t = tid; t < p.n_max; t += kThreads) {
    if (t >= P && t < n) {
      if (!((bitmap[t >> 5] >> (t & 31)) & 1u)) out[t] = (float)(-up * exp((double)s[t] - M) * c_carry);
    } else {
      out[t] = 0.f;
    }
  }
}

// ---------------------------------------------------------------- lists of at most 32 units

constexpr int kTinyWarps = 8;

__global__ void __launch_bounds__(kTinyWarps * 32) logprob_tiny_kernel(LogprobParams p, int64_t n_lists) {
  const int lane = threadIdx.x & 31;
  const int64_t li = (int64_t)blockIdx.x * kTinyWarps + (threadIdx.x >> 5);
  if (li >= n_lists) return;
  const int64_t outer = li / p.G;
  const int n = p.n[outer];
  const int P = p.n_protect ? p.n_protect[outer] : 0;
  const int K = p.budget[outer];
  const int Kp = K - P;
  const float* s = p.logits + li * p.n_max;
  const int32_t* sigma = p.kept_order + li * p.k_max;
  const double kNaN = __longlong_as_double(0x7ff8000000000000LL);

  if (!(P >= 0 && P <= K && K <= n && n <= p.n_max && Kp <= p.k_max)) {
    if (lane == 0) { set_dev_status(p.dev_status, NGC_DEV_BAD_COUNTS); p.logp[li] = kNaN; }
    return;
  }
  // lane j holds sigma_j; lane t holds logit t
  const int sj = lane < Kp ? sigma[lane] : -1;
  const bool in_range = lane >= Kp || (sj >= P && sj < n);
  uint32_t drawn = 0;                 // bit t set: unit t was drawn
  bool repeat = false;
  for (int j = 0; j < Kp; ++j) {
    const int t = __shfl_sync(0xffffffffu, sj, j) & 31;
    if (drawn & (1u << t)) repeat = true;
    drawn |= 1u << t;
  }
  if (!__all_sync(0xffffffffu, in_range) || repeat) {
    if (lane == 0) { set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT); p.logp[li] = kNaN; }
    return;
  }
  if (Kp == 0) {
    if (lane == 0) p.logp[li] = 0.0;
    return;
  }
  const bool cand = lane >= P && lane < n;
  const float v = cand ? s[lane] : -INFINITY;
  if (__any_sync(0xffffffffu, cand && v != v)) {
    if (lane == 0) { set_dev_status(p.dev_status, NGC_DEV_NAN_LOGIT); p.logp[li] = kNaN; }
    return;
  }
  const double M = (double)warp_max(v);
  const double e_t = cand ? exp((double)v - M) : 0.0;
  // mass never drawn, then the tail sums of the drawn masses in sigma order
  const double U = warp_sum(((drawn >> lane) & 1u) ? 0.0 : e_t);
  const int src = sj < 0 ? 0 : sj;
  const double z = __shfl_sync(0xffffffffu, (double)v - M, src);     // s_sigma_j - M on lane j
  const double e = __shfl_sync(0xffffffffu, e_t, src);
  double tail = lane < Kp ? e : 0.0;                                 // -> sum_{i >= j} e_sigma_i
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_down_sync(0xffffffffu, tail, o);
    if (lane + o < 32) tail += t;
  }
  const double total = warp_sum(lane < Kp ? z - log(U + tail) : 0.0);
  if (lane == 0) p.logp[li] = total;
}

__global__ void __launch_bounds__(kTinyWarps * 32) logprob_grad_tiny_kernel(GradParams g, int64_t n_lists) {
  const LogprobParams& p = g.f;
  const int lane = threadIdx.x & 31;
  const int64_t li = (int64_t)blockIdx.x * kTinyWarps + (threadIdx.x >> 5);
  if (li >= n_lists) return;
  const int64_t outer = li / p.G;
  const int n = p.n[outer];
  const int P = p.n_protect ? p.n_protect[outer] : 0;
  const int K = p.budget[outer];
  const int Kp = K - P;
  const float* s = p.logits + li * p.n_max;
  const int32_t* sigma = p.kept_order + li * p.k_max;
  float* out = g.grad_logits + li * p.n_max;
  const float kNaNf = __int_as_float(0x7fc00000);

  int fail = 0;
  int sj = -1;
  uint32_t drawn = 0;
  float v = -INFINITY;
  const bool counts_ok = P >= 0 && P <= K && K <= n && n <= p.n_max && Kp <= p.k_max;
  const bool cand = counts_ok && lane >= P && lane < n;
  if (!counts_ok) fail = NGC_DEV_BAD_COUNTS;
  if (!fail) {
    sj = lane < Kp ? sigma[lane] : -1;
    const bool in_range = lane >= Kp || (sj >= P && sj < n);
    bool repeat = false;
    for (int j = 0; j < Kp; ++j) {
      const int t = __shfl_sync(0xffffffffu, sj, j) & 31;
      if (drawn & (1u << t)) repeat = true;
      drawn |= 1u << t;
    }
    if (!__all_sync(0xffffffffu, in_range) || repeat) fail = NGC_DEV_BAD_KEPT;
  }
  if (!fail) {
    v = cand ? s[lane] : -INFINITY;
    if (__any_sync(0xffffffffu, cand && v != v)) fail = NGC_DEV_NAN_LOGIT;
  }
  if (fail) {
    if (lane == 0) set_dev_status(p.dev_status, fail);
    if (lane < p.n_max) out[lane] = kNaNf;
    return;
  }
  const double up = g.grad_logp ? g.grad_logp[li] : 1.0;
  const double M = (double)warp_max(v);                   // -inf when nothing is a candidate (then Kp = 0)
  const double e_t = cand ? exp((double)v - M) : 0.0;
  const double U = warp_sum(((drawn >> lane) & 1u) ? 0.0 : e_t);
  const int src = sj < 0 ? 0 : sj;
  const double e = __shfl_sync(0xffffffffu, e_t, src);               // e_sigma_j on lane j
  double tail = lane < Kp ? e : 0.0;                                 // -> sum_{i >= j} e_sigma_i
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_down_sync(0xffffffffu, tail, o);
    if (lane + o < 32) tail += t;
  }
  double C = lane < Kp ? 1.0 / (U + tail) : 0.0;                     // -> sum_{i <= j} 1 / rem_i
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(0xffffffffu, C, o);
    if (lane >= o) C += t;
  }
  const double C_all = __shfl_sync(0xffffffffu, C, 31);
  if (lane < p.n_max) out[lane] = cand ? (float)(-up * e_t * C_all) : 0.f;      // as if never drawn
  __syncwarp();
  if (lane < Kp) out[sj] = (float)(up * (1.0 - e * C));                         // the drawn units
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_evict_logprob(const float* logits, const int32_t* n, const int32_t* n_protect,
                                 const int32_t* budget, const int32_t* kept_order,
                                 int n_batches, int B, int G, int n_max, int k_max, double* logp,
                                 void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_evict_logprob");
  using namespace ngc;
  (void)ws; (void)ws_bytes;
  if (!logits || !n || !budget || !kept_order || !logp || n_batches <= 0 || B <= 0 || G <= 0 || n_max <= 0 || k_max <= 0)
    return NGC_ERR_INVALID_ARG;
  const int64_t lists = (int64_t)n_batches * B * G;
  if (lists > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  const size_t smem = (size_t)((n_max + 31) / 32) * 4;
  if (smem > 200 * 1024) return NGC_ERR_UNSUPPORTED;
  if (smem > 48 * 1024)
    NGC_CUDA_TRY(cudaFuncSetAttribute(logprob_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LogprobParams p;
  p.logits = logits; p.n = n; p.n_protect = n_protect; p.budget = budget; p.kept_order = kept_order;
  p.logp = logp; p.dev_status = dev_status; p.G = G; p.n_max = n_max; p.k_max = k_max;
  if (n_max <= 32)
    logprob_tiny_kernel<<<(unsigned)((lists + kTinyWarps - 1) / kTinyWarps), kTinyWarps * 32, 0, (cudaStream_t)stream>>>(p, lists);
  else
    logprob_kernel<<<(unsigned)lists, kThreads, smem, (cudaStream_t)stream>>>(p);
  return launch_status();
}

extern "C" int ngc_evict_logprob_backward(const float* logits, const int32_t* n, const int32_t* n_protect,
                                          const int32_t* budget, const int32_t* kept_order, const double* grad_logp,
                                          int n_batches, int B, int G, int n_max, int k_max, float* grad_logits,
                                          void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_evict_logprob_backward");
  using namespace ngc;
  (void)ws; (void)ws_bytes;
  if (!logits || !n || !budget || !kept_order || !grad_logits || n_batches <= 0 || B <= 0 || G <= 0 || n_max <= 0 || k_max <= 0)
    return NGC_ERR_INVALID_ARG;
  const int64_t lists = (int64_t)n_batches * B * G;
  if (lists > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  GradParams g;
  g.f.logits = logits; g.f.n = n; g.f.n_protect = n_protect; g.f.budget = budget; g.f.kept_order = kept_order;
  g.f.logp = nullptr; g.f.dev_status = dev_status; g.f.G = G; g.f.n_max = n_max; g.f.k_max = k_max;
  g.grad_logp = grad_logp; g.grad_logits = grad_logits;
  if (n_max <= 32) {
    logprob_grad_tiny_kernel<<<(unsigned)((lists + kTinyWarps - 1) / kTinyWarps), kTinyWarps * 32, 0, (cudaStream_t)stream>>>(g, lists);
    return launch_status();
  }
  const size_t smem = (size_t)(k_max < n_max ? k_max : n_max) * 8 + (size_t)((n_max + 31) / 32) * 4;
  if (smem > 200 * 1024) return NGC_ERR_UNSUPPORTED;
  if (smem > 48 * 1024)
    NGC_CUDA_TRY(cudaFuncSetAttribute(logprob_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  logprob_grad_kernel<<<(unsigned)lists, kThreads, smem, (cudaStream_t)stream>>>(g);
  return launch_status();
}
