// ngc_score_evict: attention-based eviction scores (paper Section 4.2).
//
// psi_t = mean over (query head, recent query) rows of softmax(q K^T / sqrt(d))_t,
// s_j = mean of psi over the tokens of unit j.  The softmax of a row spans the
// whole strip, so the work is split into three launches:
//   1. per (strip, token range): the row-wise max and sum of exponentials of the
//      range's scores;
//   2. same geometry: the range statistics of a row are merged, the scores are
//      recomputed and each token's probability summed over the rows of the
//      strip is written out;
//   3. per list: the strips feeding the list are added in a fixed order, the
//      block mean is taken and the logit written.
// No atomics on floating-point data: the result is reproducible run to run.
//
// Two device paths for launches 1 and 2:
//  * bf16, d = 128, at most 40 rows per strip (group size x window): the strip
//    is streamed once per launch through a TMA + mbarrier ring (64 tokens x 128
//    channels per stage, 128-byte swizzle) and S = K Q^T runs on the tensor
//    cores (mma.sync m16n8k16: 16 tokens on M, the strip's rows on N, their
//    query fragments held in registers), so the launch stays HBM-bound.
//  * everything else: a thread owns one token, the rows' queries sit in shared
//    memory as fp32, plain FMA.
#include <cuda_bf16.h>

#include "kv_map.cuh"
#include "ngc_common.cuh"
#include "ngc_plan.h"
#include "ptx.cuh"

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
  int32_t* n_units_out;   // [B] or null: units of the sequence's longest list
  float2* stats;     // [strips][n_chunks][rows] (max, sum exp)
  float* psi;        // [L*Hkv*R] per-token probability mass summed over the strip's rows
  int64_t rows_R;
  int L, B, Hq, Hkv, g, w, n_rows;   // n_rows = g * w rows per strip
  int n_chunks, block, lists, G, n_max, log_transform;
  int n_split;       // token ranges per strip (streaming path)
  float inv_sqrt_d;
  // paged layout (page_table != null): K rows of a plane = B * pages_cap * page, seq_off unused;
  // psi is indexed by logical token: sequence b starts at b * pages_cap * page
  const int32_t* page_table;   // [B][G_tab][pages_cap]
  int page, pages_cap, tab_lists, tab_G;
  int lens_lists;              // 0: lens[B]; else == lists: lens[B][G]
};

__device__ __forceinline__ int64_t psi_row0(const ScoreParams& p, int b) {
  return p.page_table ? (int64_t)b * p.pages_cap * p.page : p.seq_off[b];
}

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
  const int T_b = p.lens[len_index(p.lens_lists, p.L, p.Hkv, b, l, h)];
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

// ---------------------------------------------------------------- streaming bf16 path

constexpr int kSTileT = 64;                       // tokens per stage
constexpr int kSConsumerWarps = 4;
constexpr int kSThreads = (kSConsumerWarps + 1) * 32;
constexpr int kSBoxBytes = kSTileT * 128;         // 64 tokens x 64 channels of bf16
constexpr int kSStageBytes = 2 * kSBoxBytes;      // channels 0-63 and 64-127
constexpr int kSStages = 4;
constexpr int kSMaxRows = 40;                     // rows (columns of S) a strip may have on this path

// (m, s) <- merge of two (max, sum of 2^(z - max)) pairs; either side may be empty (m = -inf).
__device__ __forceinline__ void merge_ms(float& m, float& s, float mo, float so) {
  const float mn = fmaxf(m, mo);
  if (mn == -INFINITY) { s = 0.f; return; }
  s = s * ptx::ex2_approx(m - mn) + so * ptx::ex2_approx(mo - mn);
  m = mn;
}

// NT = number of 8-column tiles of S (ceil(rows / 8)).  PASS 1 writes the range
// statistics, PASS 2 the per-token probability mass.  Scores are kept in the
// log2 domain: z = (q.k) * scale * log2(e).
template <int NT, int PASS>
__global__ void __launch_bounds__(kSThreads, 2)
score_stream_kernel(const __grid_constant__ CUtensorMap map_k, ScoreParams p, float scale_log2, int32_t* dev_status) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ uint64_t bar_full[kSStages], bar_empty[kSStages];
  __shared__ float2 sm_ms[kSConsumerWarps][kSMaxRows];
  __shared__ float sm_M[kSMaxRows], sm_inv[kSMaxRows];

  uint8_t* stage_base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;

  const int split = blockIdx.x % p.n_split;
  const int strip = blockIdx.x / p.n_split;
  const int h = strip % p.Hkv;
  const int b = (strip / p.Hkv) % p.B;
  const int l = strip / (p.Hkv * p.B);
  const int T_b = p.lens[len_index(p.lens_lists, p.L, p.Hkv, b, l, h)];
  const int n_rows = p.n_rows;
  const int w_eff = min(p.w, T_b);

  const int nt = (T_b + kSTileT - 1) / kSTileT;
  const int tps = (nt + p.n_split - 1) / p.n_split;
  const int tile_lo = min(nt, split * tps);
  const int tile_hi = min(nt, tile_lo + tps);
  const int n_tiles = tile_hi - tile_lo;

  float2* st = p.stats + (int64_t)strip * p.n_split * kSMaxRows;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kSStages; ++s) { ptx::mbar_init(&bar_full[s], 1); ptx::mbar_init(&bar_empty[s], kSConsumerWarps); }
    ptx::fence_barrier_init();
  }
  if (PASS == 2 && tid < kSMaxRows) {
    float m = -INFINITY, sum = 0.f;
    for (int c = 0; c < p.n_split; ++c) {
      const float2 v = st[c * kSMaxRows + tid];
      merge_ms(m, sum, v.x, v.y);
    }
    const bool live = tid < n_rows && sum > 0.f;
    sm_M[tid] = live ? m : 0.f;
    sm_inv[tid] = live ? 1.f / sum : 0.f;
  }
  __syncthreads();

  if (warp == kSConsumerWarps) {
    // ------------------------------------------------ producer
    if (lane == 0 && n_tiles > 0) {
      ptx::prefetch_tensormap(&map_k);
      const int plane = l * p.Hkv + h;
      const int32_t* table = p.page_table
          ? p.page_table + ((int64_t)b * p.tab_G + list_of(p.tab_lists, l, h, p.Hkv)) * p.pages_cap : nullptr;
      const int row0 = table ? 0 : (int)p.seq_off[b];
      const int n_sub = table ? kSTileT / p.page : 1;          // pages per 64-token tile
      const int sub_bytes = (kSTileT / n_sub) * 128;
      for (int it = 0; it < n_tiles; ++it) {
        const int s = it % kSStages;
        if (it >= kSStages) {
          if (!ptx::mbar_wait_bounded(&bar_empty[s], ((it / kSStages) - 1) & 1)) set_dev_status(dev_status, NGC_DEV_TIMEOUT);
        }
        uint8_t* sp = stage_base + s * kSStageBytes;
        ptx::mbar_expect_tx(&bar_full[s], kSStageBytes);
        for (int sb = 0; sb < n_sub; ++sb) {
          int y;
          if (table) {
            const int j = min(p.pages_cap - 1, (tile_lo + it) * n_sub + sb);   // free pages are mapped too
            y = (b * p.pages_cap + table[j]) * p.page;
          } else {
            y = row0 + (tile_lo + it) * kSTileT;
          }
          // the first row of a tile holds a live token (a box that overhangs the plane reads zeros)
          if (!NGC_IN_BOUNDS(dev_status, y >= 0 && y < p.rows_R)) y = 0;
          ptx::tma_load_3d(sp + sb * sub_bytes, &map_k, 0, y, plane, &bar_full[s]);
          ptx::tma_load_3d(sp + sb * sub_bytes + kSBoxBytes, &map_k, 64, y, plane, &bar_full[s]);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ consumers
    // B operand: Q^T, column n of an 8-wide tile = row 8*tile + n of the strip
    // (row r = head-in-group r / w, window slot r % w); zero beyond n_rows.
    uint32_t qb[NT][8][2];
    int lim[NT][2];          // last visible token of the thread's columns (-1: column unused)
#pragma unroll
    for (int t8 = 0; t8 < NT; ++t8) {
      const int r = 8 * t8 + gid;
      const bool live = r < n_rows;
      const int hl = live ? r / p.w : 0, j = live ? r - hl * p.w : 0;
      const uint32_t* qrow = (const uint32_t*)((const __nv_bfloat16*)p.q_recent +
                                               ((((int64_t)l * p.B + b) * p.Hq + h * p.g + hl) * p.w + j) * 128);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[t8][ks][0] = live ? qrow[8 * ks + tig] : 0u;
        qb[t8][ks][1] = live ? qrow[8 * ks + tig + 4] : 0u;
      }
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int c = 8 * t8 + 2 * tig + e;
        const int jc = c % p.w;
        // window slot j sits at absolute position T_b - w + j; slots before the sequence start do not exist
        lim[t8][e] = (c < n_rows && jc >= p.w - w_eff) ? T_b - p.w + jc : -1;
      }
    }
    float m_run[NT][2], s_run[NT][2];      // PASS 1: running max (raw dot products) and sum
    float negM[NT][2], inv[NT][2];         // PASS 2: -M (log2 domain) and 1 / row sum
#pragma unroll
    for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        m_run[t8][e] = -INFINITY; s_run[t8][e] = 0.f;
        if (PASS == 2) {
          const int c = 8 * t8 + 2 * tig + e;
          negM[t8][e] = -sm_M[c];
          inv[t8][e] = sm_inv[c];
        } else {
          negM[t8][e] = 0.f; inv[t8][e] = 0.f;
        }
      }
    const uint32_t a_lane_off = (uint32_t)((16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * 128);
    const uint32_t x7 = (uint32_t)(lane & 7);
    float* psi_strip = p.psi + (int64_t)(l * p.Hkv + h) * p.rows_R + psi_row0(p, b);

    for (int it = 0; it < n_tiles; ++it) {
      const int s = it % kSStages;
      if (!ptx::mbar_wait_bounded(&bar_full[s], (it / kSStages) & 1)) set_dev_status(dev_status, NGC_DEV_TIMEOUT);
      const uint32_t k_st = ptx::smem_u32(stage_base + s * kSStageBytes);
      const int t_base = (tile_lo + it) * kSTileT + 16 * warp;

      if (t_base < T_b) {
        float acc[NT][4];
#pragma unroll
        for (int t8 = 0; t8 < NT; ++t8) { acc[t8][0] = 0.f; acc[t8][1] = 0.f; acc[t8][2] = 0.f; acc[t8][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t chunk = (uint32_t)(2 * (ks & 3) + (lane >> 4));
          const uint32_t addr = k_st + (ks >> 2) * kSBoxBytes + a_lane_off + ((chunk ^ x7) << 4);
          uint32_t a[4];
          ptx::ldmatrix_x4(addr, a[0], a[1], a[2], a[3]);
#pragma unroll
          for (int t8 = 0; t8 < NT; ++t8) ptx::mma_bf16_16816(acc[t8], a, qb[t8][ks][0], qb[t8][ks][1]);
        }
        const int t0 = t_base + gid, t1 = t0 + 8;
        // tokens of this slice that some row cannot see: the window itself and the tail beyond T_b
        const bool masked = t_base + 16 > T_b - p.w;
        if (PASS == 1) {
#pragma unroll
          for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float a0 = acc[t8][e], a1 = acc[t8][e + 2];
              if (masked) {
                a0 = t0 <= lim[t8][e] ? a0 : -INFINITY;
                a1 = t1 <= lim[t8][e] ? a1 : -INFINITY;
              }
              const float mx = fmaxf(fmaxf(m_run[t8][e], a0), a1);
              const float ms = masked && mx == -INFINITY ? 0.f : mx;
              const float neg = -ms * scale_log2;
              const float e_old = ptx::ex2_approx(fmaf(m_run[t8][e], scale_log2, neg));
              const float e0 = ptx::ex2_approx(fmaf(a0, scale_log2, neg));
              const float e1 = ptx::ex2_approx(fmaf(a1, scale_log2, neg));
              s_run[t8][e] = fmaf(s_run[t8][e], e_old, e0 + e1);
              m_run[t8][e] = mx;
            }
        } else {
          float p0 = 0.f, p1 = 0.f;
#pragma unroll
          for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float e0 = ptx::ex2_approx(fmaf(acc[t8][e], scale_log2, negM[t8][e]));
              float e1 = ptx::ex2_approx(fmaf(acc[t8][e + 2], scale_log2, negM[t8][e]));
              if (masked) {
                e0 = t0 <= lim[t8][e] ? e0 : 0.f;
                e1 = t1 <= lim[t8][e] ? e1 : 0.f;
              }
              p0 = fmaf(e0, inv[t8][e], p0);
              p1 = fmaf(e1, inv[t8][e], p1);
            }
          p0 += __shfl_xor_sync(0xffffffffu, p0, 1);
          p0 += __shfl_xor_sync(0xffffffffu, p0, 2);
          p1 += __shfl_xor_sync(0xffffffffu, p1, 1);
          p1 += __shfl_xor_sync(0xffffffffu, p1, 2);
          if (tig == 0 && NGC_IN_BOUNDS(dev_status, psi_row0(p, b) + t1 < p.rows_R || t1 >= T_b)) {
            if (t0 < T_b) psi_strip[t0] = p0;
            if (t1 < T_b) psi_strip[t1] = p1;
          }
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&bar_empty[s]);
    }
    if (PASS == 1) {
      // columns are spread over the quad (tig), tokens over gid: merge over gid, then over warps
#pragma unroll
      for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          float m = m_run[t8][e] * scale_log2, sum = s_run[t8][e];     // -inf stays -inf (scale > 0)
#pragma unroll
          for (int o = 4; o < 32; o <<= 1) {
            const float mo = __shfl_xor_sync(0xffffffffu, m, o);
            const float so = __shfl_xor_sync(0xffffffffu, sum, o);
            merge_ms(m, sum, mo, so);
          }
          if (gid == 0) sm_ms[warp][8 * t8 + 2 * tig + e] = make_float2(m, sum);
        }
    }
  }
  if (PASS == 1) {
    __syncthreads();
    if (tid < kSMaxRows) {
      float m = -INFINITY, sum = 0.f;
      if (tid < 8 * NT) {
#pragma unroll
        for (int w2 = 0; w2 < kSConsumerWarps; ++w2) merge_ms(m, sum, sm_ms[w2][tid].x, sm_ms[w2][tid].y);
      }
      st[split * kSMaxRows + tid] = make_float2(m, sum);
    }
  }
}

// ---------------------------------------------------------------- list reduction

__global__ void __launch_bounds__(256) score_finish_kernel(ScoreParams p) {
  __shared__ int s_seq_units;
  const int li = blockIdx.x;                    // b * G + gi
  const int b = li / p.G, gi = li - b * p.G;
  const int T_b = p.lens[p.lens_lists ? li : b];      // a length per list means lens_lists == lists
  const int n_units = (T_b + p.block - 1) / p.block;
  // units of the sequence's longest list: with a length per list the sampler works on that many units per
  // sequence, and the units a shorter list does not have must carry logit -inf (never drawn, no mass in Eq. (1))
  int seq_units = n_units;
  if (p.lens_lists) {
    if (threadIdx.x == 0) s_seq_units = 0;
    __syncthreads();
    for (int g2 = threadIdx.x; g2 < p.G; g2 += blockDim.x)
      atomicMax(&s_seq_units, (p.lens[(int64_t)b * p.G + g2] + p.block - 1) / p.block);
    __syncthreads();
    seq_units = s_seq_units;
  }
  if (p.n_units_out && gi == 0 && blockIdx.y == 0 && threadIdx.x == 0) p.n_units_out[b] = seq_units;
  const int u = blockIdx.y * blockDim.x + threadIdx.x;
  if (u >= p.n_max) return;
  if (u >= n_units) {
    if (u < seq_units) p.logits[(int64_t)li * p.n_max + u] = -INFINITY;
    return;
  }
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
      for (int h = h0; h < h1; ++h) m += p.psi[(int64_t)(l * p.Hkv + h) * p.rows_R + psi_row0(p, b) + t];
    acc += m / n_rows_list;
  }
  const float s = acc / (float)(t1 - t0);
  p.logits[(int64_t)li * p.n_max + u] = p.log_transform ? logf(s) : s;
}

constexpr int kScoreTargetCtas = 148 * 2 * 2;   // two waves of two CTAs per SM

bool score_stream_shape(const ngc_cache* c, int w) {
  return c->dtype == NGC_BF16 && c->d == 128 && (c->Hq / c->Hkv) * w <= kSMaxRows && c->rows < 0x7fffffffLL;
}

// Token ranges per strip on the streaming path: enough CTAs to fill the GPU, at least 4 tiles each.
int score_n_split(const ngc_cache* c) {
  const int64_t strips = (int64_t)c->L * c->B * c->Hkv;
  if (strips >= kScoreTargetCtas) return 1;
  int ns = (int)((kScoreTargetCtas + strips - 1) / strips);
  const int by_len = (c->max_len + 4 * kSTileT - 1) / (4 * kSTileT);
  if (ns > by_len) ns = by_len;
  if (ns > 64) ns = 64;
  return ns < 1 ? 1 : ns;
}

size_t stats_bytes(const ngc_cache* c) {
  const int n_chunks = (c->max_len + kChunk - 1) / kChunk;
  const size_t strips = (size_t)c->L * c->Hkv * c->B;
  const size_t generic = strips * (n_chunks > 0 ? n_chunks : 1) * (c->Hq / c->Hkv) * 16 /*w <= 16*/ * 8;
  const size_t stream = strips * score_n_split(c) * kSMaxRows * 8;
  return align256(generic > stream ? generic : stream);
}

template <int NT>
int launch_score_stream(const CUtensorMap& map_k, const ScoreParams& p, float scale_log2, int32_t* dev_status,
                        unsigned grid, cudaStream_t stream) {
  const int smem = kSStages * kSStageBytes + 1024;
  static PerDeviceOnce attr_once;      // the shared-memory opt-in is stored per device
  const int attr_rc = attr_once.run([&] {
    cudaError_t e = cudaFuncSetAttribute(score_stream_kernel<NT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_stream_kernel<NT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return e;
  });
  if (attr_rc != NGC_OK) return attr_rc;
  score_stream_kernel<NT, 1><<<grid, kSThreads, smem, stream>>>(map_k, p, scale_log2, dev_status);
  score_stream_kernel<NT, 2><<<grid, kSThreads, smem, stream>>>(map_k, p, scale_log2, dev_status);
  return launch_status();
}

}  // namespace

size_t score_workspace_bytes(const ngc_cache* c, int G, int n_max) {
  (void)G; (void)n_max;
  return align256((size_t)c->L * c->Hkv * c->rows * 4) + stats_bytes(c);
}

}  // namespace ngc

namespace ngc {
namespace {

int score_impl(const ngc_cache* c, const PagedView& pv, const void* q_recent, int w, int block, int lists,
               int log_transform, float* logits, int n_max, int32_t* n_units_out,
               void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t stream) {
  if (!q_recent || !logits || w <= 0 || w > 16 || block <= 0 || lists < 0 || lists > 2 || n_max <= 0)
    return NGC_ERR_INVALID_ARG;
  const int g = c->Hq / c->Hkv;
  if (g * w > 128) return NGC_ERR_UNSUPPORTED;
  if (c->lens_lists != 0 && c->lens_lists != lists) return NGC_ERR_INVALID_ARG;   // a length per scored list, or one per sequence
  if ((int64_t)n_max * block < c->max_len) return NGC_ERR_INVALID_ARG;
  if (c->rows == 0 || c->max_len == 0) return NGC_OK;
  const size_t need = score_workspace_bytes(c, 0, n_max);
  if (!ws || ws_bytes < need || ((uintptr_t)ws & 255)) return NGC_ERR_WORKSPACE;

  ScoreParams p;
  p.k = c->k; p.q_recent = q_recent; p.seq_off = c->seq_off; p.lens = c->lens; p.logits = logits;
  p.n_units_out = n_units_out;
  p.psi = (float*)ws;
  p.stats = (float2*)((char*)ws + align256((size_t)c->L * c->Hkv * c->rows * 4));
  p.rows_R = c->rows;
  p.L = c->L; p.B = c->B; p.Hq = c->Hq; p.Hkv = c->Hkv; p.g = g; p.w = w; p.n_rows = g * w;
  p.n_chunks = (c->max_len + kChunk - 1) / kChunk;
  p.block = block; p.lists = lists; p.G = lists_G(lists, c->L, c->Hkv); p.n_max = n_max;
  p.log_transform = log_transform;
  p.inv_sqrt_d = 1.0f / sqrtf((float)c->d);
  p.page_table = pv.table; p.page = pv.page; p.pages_cap = pv.pages_cap; p.tab_lists = pv.lists;
  p.lens_lists = c->lens_lists;
  p.tab_G = lists_G(pv.lists, c->L, c->Hkv);

  p.n_split = 1;
  int rc;
  const bool stream_ok = score_stream_shape(c, w) && ((uintptr_t)c->k & 15) == 0 && ((uintptr_t)q_recent & 3) == 0;
  if (pv.table && !stream_ok) return NGC_ERR_UNSUPPORTED;      // paged caches: bf16, d = 128, at most 40 rows per strip
  if (stream_ok) {
    p.n_split = score_n_split(c);
    const int64_t ctas = (int64_t)c->L * c->B * c->Hkv * p.n_split;
    if (ctas > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
    CUtensorMap map_k;
    if (!make_kv_map(&map_k, c->k, c->rows, c->L * c->Hkv, pv.table ? pv.page : kSTileT)) return NGC_ERR_UNSUPPORTED;
    const float scale_log2 = p.inv_sqrt_d * 1.4426950408889634f;
    const unsigned grid = (unsigned)ctas;
    switch ((p.n_rows + 7) / 8) {
      case 1: rc = launch_score_stream<1>(map_k, p, scale_log2, dev_status, grid, stream); break;
      case 2: rc = launch_score_stream<2>(map_k, p, scale_log2, dev_status, grid, stream); break;
      case 3: rc = launch_score_stream<3>(map_k, p, scale_log2, dev_status, grid, stream); break;
      case 4: rc = launch_score_stream<4>(map_k, p, scale_log2, dev_status, grid, stream); break;
      default: rc = launch_score_stream<5>(map_k, p, scale_log2, dev_status, grid, stream); break;
    }
  } else {
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
    rc = launch_status();
  }
  if (rc != NGC_OK) return rc;
  const int n_units_max = (c->max_len + block - 1) / block;
  dim3 fgrid(c->B * p.G, (n_units_max + 255) / 256);
  if (fgrid.y > 65535) return NGC_ERR_UNSUPPORTED;
  score_finish_kernel<<<fgrid, 256, 0, stream>>>(p);
  return launch_status();
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_score_evict_launches(const ngc_cache* c, int w) {
  using namespace ngc;
  if (!valid_cache(c) || w <= 0 || c->rows == 0 || c->max_len == 0) return 0;
  return 3;      // statistics, probabilities, list reduction
}

extern "C" int ngc_score_evict(const ngc_cache* c, const void* q_recent, int w, int block, int lists,
                               int log_transform, float* logits, int n_max, int32_t* n_units_out,
                               void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_score_evict");
  using namespace ngc;
  if (!valid_cache(c)) return NGC_ERR_INVALID_ARG;
  const PagedView none = {nullptr, 0, 0, NGC_LISTS_SHARED};
  return score_impl(c, none, q_recent, w, block, lists, log_transform, logits, n_max, n_units_out, ws, ws_bytes, dev_status,
                    (cudaStream_t)stream);
}

extern "C" int ngc_score_evict_paged(const ngc_paged_cache* pc, const void* q_recent, int w, int log_transform,
                                     float* logits, int n_max, int32_t* n_units_out, void* ws, size_t ws_bytes,
                                     int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_score_evict_paged");
  using namespace ngc;
  if (!pc || !pc->k || !pc->page_table || !pc->lens || pc->L <= 0 || pc->B <= 0 || pc->Hq <= 0 || pc->Hkv <= 0 ||
      pc->Hq % pc->Hkv != 0 || pc->pages_cap <= 0 || (pc->page != 32 && pc->page != 64) || pc->lists < 0 || pc->lists > 2)
    return NGC_ERR_INVALID_ARG;
  if (pc->dtype != NGC_BF16 || pc->d != 128) return NGC_ERR_UNSUPPORTED;
  ngc_cache c;
  c.k = pc->k; c.v = pc->v; c.seq_off = nullptr; c.lens = pc->lens;
  c.rows = (int64_t)pc->B * pc->pages_cap * pc->page;
  c.L = pc->L; c.B = pc->B; c.Hq = pc->Hq; c.Hkv = pc->Hkv; c.d = pc->d; c.dtype = pc->dtype;
  c.max_len = pc->pages_cap * pc->page;
  c.lens_lists = pc->lens_per_list ? pc->lists : 0;
  const PagedView pv = {pc->page_table, pc->page, pc->pages_cap, pc->lists};
  return score_impl(&c, pv, q_recent, w, pc->page, pc->lists, log_transform, logits, n_max, n_units_out, ws, ws_bytes,
                    dev_status, (cudaStream_t)stream);
}
