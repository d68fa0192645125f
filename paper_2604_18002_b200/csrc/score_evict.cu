// ngc_score_evict: attention-based eviction scores (paper Section 4.2).
//
// psi_t = mean over (query head, recent query) rows of softmax(q K^T / sqrt(d))_t,
// s_j = mean of psi over the tokens of unit j.  The softmax of a row spans the
// whole strip, so the work is split into three launches:
//   1. per (strip, 256-token chunk): the row-wise max and sum of exponentials
//      of the chunk's scores (a thread owns one token, the rows' queries sit in
//      shared memory as fp32);
//   2. same geometry: the chunk statistics of a row are merged, the scores are
//      recomputed (K comes from L2 where it fits) and each token's probability
//      summed over the rows of the strip is written out;
//   3. per list: the strips feeding the list are added in a fixed order, the
//      block mean is taken and the logit written.
// No atomics on floating-point data: the result is reproducible run to run.
#include <cuda_bf16.h>

#include "ngc_common.cuh"
#include "ngc_plan.h"

namespace ngc {
namespace {

constexpr int kChunk = 256;     // tokens per CTA == threads per CTA
constexpr int kRowTile = 8;     // rows scored per pass over a K row
constexpr int kWarps = kChunk / 32;

struct ScoreParams {
  const void* k;
  const void* q_recent;
  const int64_t* seq_off;
  const int32_t* lens;
  float* logits;
  float2* stats;     // [strips][n_chunks][rows] (max, sum exp)
  float* psi;        // [L*Hkv*R] per-token probability mass summed over the strip's rows
  int64_t rows_R;
  int L, B, Hq, Hkv, g, w, n_rows;   // n_rows = g * w rows per strip
  int n_chunks, block, lists, G, n_max, log_transform;
  float inv_sqrt_d;
};

template <typename T> __device__ __forceinline__ void load8(const T* p, float (&x)[8]);
template <> __device__ __forceinline__ void load8<float>(const float* p, float (&x)[8]) {
  const float4 a = ((const float4*)p)[0], b = ((const float4*)p)[1];
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
template <> __device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&x)[8]) {
  const uint4 a = *(const uint4*)p;
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(w[i] << 16);
    x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T, int D, int PASS>
__global__ void __launch_bounds__(kChunk) score_kernel(ScoreParams p) {
  extern __shared__ float qs[];                 // [n_rows][D]
  __shared__ float s_redm[kWarps][kRowTile], s_reds[kWarps][kRowTile];
  __shared__ float s_rowm[128], s_rowinv[128];  // merged row statistics (PASS 2)

  const int chunk = blockIdx.x % p.n_chunks;
  int strip = blockIdx.x / p.n_chunks;
  const int h = strip % p.Hkv;
  const int b = (strip / p.Hkv) % p.B;
  const int l = strip / (p.Hkv * p.B);
  const int T_b = p.lens[b];
  if (chunk * kChunk >= T_b) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = chunk * kChunk + tid;
  const bool active = t < T_b;
  const int w_eff = min(p.w, T_b);
  const int n_rows = p.n_rows;

  // queries of the strip's rows -> shared, fp32.  row r = (head-in-group, window slot)
  for (int i = tid; i < n_rows * D; i += kChunk) {
    const int r = i / D, c = i - r * D;
    const int hl = r / p.w, j = r - hl * p.w;
    const T* qp = (const T*)p.q_recent + ((((int64_t)l * p.B + b) * p.Hq + h * p.g + hl) * p.w + j) * D;
    qs[i] = to_float<T>(qp[c]);
  }
  const float2* st = p.stats + ((int64_t)strip * p.n_chunks) * n_rows;
  if (PASS == 2) {
    const int n_live = (T_b + kChunk - 1) / kChunk;
    for (int r = tid; r < n_rows; r += kChunk) {
      float m = -INFINITY;
      for (int c = 0; c < n_live; ++c) m = fmaxf(m, st[(int64_t)c * n_rows + r].x);
      float sum = 0.f;
      for (int c = 0; c < n_live; ++c) {
        const float2 v = st[(int64_t)c * n_rows + r];
        if (v.x != -INFINITY) sum += v.y * expf(v.x - m);
      }
      s_rowm[r] = m;
      s_rowinv[r] = sum > 0.f ? 1.f / sum : 0.f;
    }
  }
  __syncthreads();

  const T* krow = (const T*)p.k + ((int64_t)(l * p.Hkv + h) * p.rows_R + p.seq_off[b] + (active ? t : 0)) * D;
  float mass = 0.f;
  for (int r0 = 0; r0 < n_rows; r0 += kRowTile) {
    float z[kRowTile];
#pragma unroll
    for (int i = 0; i < kRowTile; ++i) z[i] = 0.f;
    if (active) {
#pragma unroll 4
      for (int c = 0; c < D; c += 8) {
        float kx[8];
        load8<T>(krow + c, kx);
#pragma unroll
        for (int i = 0; i < kRowTile; ++i) {
          if (r0 + i < n_rows) {
            const float4 qa = *(const float4*)&qs[(r0 + i) * D + c];
            const float4 qb = *(const float4*)&qs[(r0 + i) * D + c + 4];
            float a = z[i];
            a = fmaf(kx[0], qa.x, a); a = fmaf(kx[1], qa.y, a); a = fmaf(kx[2], qa.z, a); a = fmaf(kx[3], qa.w, a);
            a = fmaf(kx[4], qb.x, a); a = fmaf(kx[5], qb.y, a); a = fmaf(kx[6], qb.z, a); a = fmaf(kx[7], qb.w, a);
            z[i] = a;
          }
        }
      }
    }
    bool vis[kRowTile];
#pragma unroll
    for (int i = 0; i < kRowTile; ++i) {
      const int r = r0 + i;
      const int j = r % p.w;
      // window slot j sits at absolute position T_b - w + j; slots before the sequence start do not exist
      vis[i] = active && r < n_rows && j >= p.w - w_eff && t <= T_b - p.w + j;
      z[i] = vis[i] ? z[i] * p.inv_sqrt_d : -INFINITY;
    }
    if (PASS == 1) {
      float m[kRowTile];
#pragma unroll
      for (int i = 0; i < kRowTile; ++i) m[i] = warp_max(z[i]);
      __syncthreads();                       // previous row tile is done with the scratch
      if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kRowTile; ++i) s_redm[warp][i] = m[i];
      }
      __syncthreads();
#pragma unroll
      for (int i = 0; i < kRowTile; ++i) {
        float mm = s_redm[0][i];
#pragma unroll
        for (int w2 = 1; w2 < kWarps; ++w2) mm = fmaxf(mm, s_redm[w2][i]);
        m[i] = mm;
      }
      float e[kRowTile];
#pragma unroll
      for (int i = 0; i < kRowTile; ++i) e[i] = warp_sum(vis[i] ? expf(z[i] - m[i]) : 0.f);
      if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kRowTile; ++i) s_reds[warp][i] = e[i];
      }
      __syncthreads();
      if (tid < kRowTile && r0 + tid < n_rows) {
        float mm = s_redm[0][tid], sum = 0.f;
#pragma unroll
        for (int w2 = 1; w2 < kWarps; ++w2) mm = fmaxf(mm, s_redm[w2][tid]);
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) sum += s_reds[w2][tid];
        const_cast<float2*>(st)[(int64_t)chunk * n_rows + r0 + tid] = make_float2(mm, sum);
      }
    } else {
#pragma unroll
      for (int i = 0; i < kRowTile; ++i)
        if (vis[i]) mass += expf(z[i] - s_rowm[r0 + i]) * s_rowinv[r0 + i];
    }
  }
  if (PASS == 2 && active) p.psi[(int64_t)(l * p.Hkv + h) * p.rows_R + p.seq_off[b] + t] = mass;
}

__global__ void __launch_bounds__(256) score_finish_kernel(ScoreParams p) {
  const int li = blockIdx.x;                    // b * G + gi
  const int b = li / p.G, gi = li - b * p.G;
  const int T_b = p.lens[b];
  const int n_units = (T_b + p.block - 1) / p.block;
  const int u = blockIdx.y * blockDim.x + threadIdx.x;
  if (u >= n_units || u >= p.n_max) return;
  int l0, l1, h0, h1;
  if (p.lists == NGC_LISTS_SHARED) { l0 = 0; l1 = p.L; h0 = 0; h1 = p.Hkv; }
  else if (p.lists == NGC_LISTS_PER_LAYER) { l0 = gi; l1 = gi + 1; h0 = 0; h1 = p.Hkv; }
  else { l0 = gi / p.Hkv; l1 = l0 + 1; h0 = gi % p.Hkv; h1 = h0 + 1; }
  const int w_eff = min(p.w, T_b);
  const float n_rows_list = (float)((l1 - l0) * (h1 - h0) * p.g * w_eff);
  const int t0 = u * p.block, t1 = min(t0 + p.block, T_b);
  float acc = 0.f;
  for (int t = t0; t < t1; ++t) {
    float m = 0.f;
    for (int l = l0; l < l1; ++l)
      for (int h = h0; h < h1; ++h) m += p.psi[(int64_t)(l * p.Hkv + h) * p.rows_R + p.seq_off[b] + t];
    acc += m / n_rows_list;
  }
  const float s = acc / (float)(t1 - t0);
  p.logits[(int64_t)li * p.n_max + u] = p.log_transform ? logf(s) : s;
}

size_t stats_bytes(const ngc_cache* c) {
  const int n_chunks = (c->max_len + kChunk - 1) / kChunk;
  return align256((size_t)c->L * c->Hkv * c->B * (n_chunks > 0 ? n_chunks : 1) * (c->Hq / c->Hkv) * 16 /*w <= 16*/ * 8);
}

}  // namespace

size_t score_workspace_bytes(const ngc_cache* c, int G, int n_max) {
  (void)G; (void)n_max;
  return align256((size_t)c->L * c->Hkv * c->rows * 4) + stats_bytes(c);
}

}  // namespace ngc

extern "C" int ngc_score_evict(const ngc_cache* c, const void* q_recent, int w, int block, int lists,
                               int log_transform, float* logits, int n_max,
                               void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream_) {
  using namespace ngc;
  (void)dev_status;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!valid_cache(c) || !q_recent || !logits || w <= 0 || w > 16 || block <= 0 || lists < 0 || lists > 2 || n_max <= 0)
    return NGC_ERR_INVALID_ARG;
  const int g = c->Hq / c->Hkv;
  if (g * w > 128) return NGC_ERR_UNSUPPORTED;
  if ((int64_t)n_max * block < c->max_len) return NGC_ERR_INVALID_ARG;
  if (c->rows == 0 || c->max_len == 0) return NGC_OK;
  const size_t need = score_workspace_bytes(c, 0, n_max);
  if (!ws || ws_bytes < need || ((uintptr_t)ws & 255)) return NGC_ERR_WORKSPACE;

  ScoreParams p;
  p.k = c->k; p.q_recent = q_recent; p.seq_off = c->seq_off; p.lens = c->lens; p.logits = logits;
  p.psi = (float*)ws;
  p.stats = (float2*)((char*)ws + align256((size_t)c->L * c->Hkv * c->rows * 4));
  p.rows_R = c->rows;
  p.L = c->L; p.B = c->B; p.Hq = c->Hq; p.Hkv = c->Hkv; p.g = g; p.w = w; p.n_rows = g * w;
  p.n_chunks = (c->max_len + kChunk - 1) / kChunk;
  p.block = block; p.lists = lists; p.G = lists_G(lists, c->L, c->Hkv); p.n_max = n_max;
  p.log_transform = log_transform;
  p.inv_sqrt_d = 1.0f / sqrtf((float)c->d);

  const int64_t ctas = (int64_t)c->L * c->B * c->Hkv * p.n_chunks;
  if (ctas > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  const size_t smem = (size_t)p.n_rows * c->d * 4;
  const unsigned grid = (unsigned)ctas;

#define NGC_SCORE_LAUNCH(T, D)                                                                                   \
  do {                                                                                                           \
    if (smem > 48 * 1024) {                                                                                      \
      NGC_CUDA_TRY(cudaFuncSetAttribute(score_kernel<T, D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
      NGC_CUDA_TRY(cudaFuncSetAttribute(score_kernel<T, D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
    }                                                                                                            \
    score_kernel<T, D, 1><<<grid, kChunk, smem, stream>>>(p);                                                    \
    score_kernel<T, D, 2><<<grid, kChunk, smem, stream>>>(p);                                                    \
  } while (0)

  if (c->dtype == NGC_F32 && c->d == 64) NGC_SCORE_LAUNCH(float, 64);
  else if (c->dtype == NGC_F32) NGC_SCORE_LAUNCH(float, 128);
  else if (c->d == 64) NGC_SCORE_LAUNCH(__nv_bfloat16, 64);
  else NGC_SCORE_LAUNCH(__nv_bfloat16, 128);
#undef NGC_SCORE_LAUNCH
  int rc = launch_status();
  if (rc != NGC_OK) return rc;
  const int n_units_max = (c->max_len + block - 1) / block;
  dim3 fgrid(c->B * p.G, (n_units_max + 255) / 256);
  if (fgrid.y > 65535) return NGC_ERR_UNSUPPORTED;
  score_finish_kernel<<<fgrid, 256, 0, stream>>>(p);
  return launch_status();
}
