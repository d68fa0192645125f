// ngc_score_evict_backward: gradient of the eviction scores (paper Section 4.2) with respect to
// the recent queries and the keys -- the path on which the eviction loss of Section 4.4 reaches
// the model (Section 4.5 recomputes the scores on the autograd graph for exactly this).
//
// With P[t] = grad_logits[unit(t)] / |unit(t)| / n_rows (the same for every attention row r of the
// list; also divided by the unit's score when the logit is log s), A = softmax rows, c[r] = sum_t
// A[r][t] P[t]:
//   dz[r][t] = A[r][t] (P[t] - c[r]) / sqrt(d),   dq[r] = sum_t dz[r][t] k[t],   dk[t] = sum_r dz[r][t] q[r].
//
// bf16, d = 128, at most 40 rows per strip (the shapes of the streaming forward kernel).  Two
// launches stream K through the same TMA + mbarrier ring as the forward pass:
//   1. per (strip, token range): row max, sum of exponentials and sum of exponentials times P;
//   2. same geometry: the merged statistics give A and c; S^T = K Q^T is
//      recomputed on the tensor cores, dz formed in registers, then
//        dK  (16 tokens x 128 channels per warp) = dZ Q          -- A operand straight from the
//                                                                   accumulators, written out as bf16;
//        dQ  (rows x 32 channels per warp)       += dZ^T K        -- dZ of the whole 64-token tile
//                                                                   exchanged through shared memory.
//      Per-range dQ partials go to the workspace; a third small kernel adds the ranges of a strip
//      in a fixed order (no float atomics: results are reproducible).
#include <cuda_bf16.h>
#include <stdlib.h>


#include "kv_map.cuh"
#include "ngc_common.cuh"
#include "ngc_plan.h"
#include "ptx.cuh"
#include "score_backward.cuh"

namespace ngc {
namespace {

constexpr int kTileT = 64;                        // tokens per stage
constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kBoxBytes = kTileT * 128;           // 64 tokens x 64 channels of bf16
constexpr int kStageBytes = 2 * kBoxBytes;
constexpr int kStagesA = 4;                       // statistics pass, two CTAs per SM
constexpr int kStagesB = 4;                       // gradient pass, two CTAs per SM
constexpr int kMaxRows = kBwdMaxRows;
constexpr int kQRowBytes = 272;                   // query row in shared memory: 256 bytes + 16 (conflict-free ldmatrix)
constexpr int kQBytes = 48 * kQRowBytes;          // rows padded to 48 (three 16-row MMA steps)
constexpr int kDzRowBytes = 112;                  // dz row (one token, 48 rows of bf16 = 96 bytes) + 16
constexpr int kDzBytes = kTileT * kDzRowBytes;

// Item decoding and token range shared by both passes.
struct Item { int split, strip, h, b, l, T_b, tile_lo, n_tiles, gi; };
__device__ __forceinline__ Item decode_item(const BwdParams& p) {
  Item it;
  it.split = blockIdx.x % p.n_split;
  it.strip = blockIdx.x / p.n_split;
  it.h = it.strip % p.Hkv;
  it.b = (it.strip / p.Hkv) % p.B;
  it.l = it.strip / (p.Hkv * p.B);
  it.T_b = p.lens[len_index(p.lens_lists, p.L, p.Hkv, it.b, it.l, it.h)];
  const int nt = (it.T_b + kTileT - 1) / kTileT;
  const int tps = (nt + p.n_split - 1) / p.n_split;
  it.tile_lo = min(nt, it.split * tps);
  it.n_tiles = min(nt, it.tile_lo + tps) - it.tile_lo;
  it.gi = list_of(p.lists, it.l, it.h, p.Hkv);
  return it;
}

// The TMA producer of both passes: K tiles of the item's token range into a ring of kNStages.
template <int kNStages>
__device__ __forceinline__ void produce_k_tiles(const CUtensorMap* map_k, const BwdParams& p, const Item& it, uint8_t* stage_base,
                                                uint64_t* bar_full, uint64_t* bar_empty) {
  ptx::prefetch_tensormap(map_k);
  const int plane = it.l * p.Hkv + it.h;
  const int row0 = (int)p.seq_off[it.b];
  for (int i = 0; i < it.n_tiles; ++i) {
    const int s = i % kNStages;
    if (i >= kNStages) {
      if (!ptx::mbar_wait_bounded(&bar_empty[s], ((i / kNStages) - 1) & 1)) set_dev_status(p.dev_status, NGC_DEV_TIMEOUT);
    }
    uint8_t* sp = stage_base + s * kStageBytes;
    ptx::mbar_expect_tx(&bar_full[s], kStageBytes);
    const int y = row0 + (it.tile_lo + i) * kTileT;
    ptx::tma_load_3d(sp, map_k, 0, y, plane, &bar_full[s]);
    ptx::tma_load_3d(sp + kBoxBytes, map_k, 64, y, plane, &bar_full[s]);
  }
}

// ---------------------------------------------------------------- pass 1: row statistics

template <int NT>
__global__ void __launch_bounds__(kThreads, 2)
score_bwd_stats_kernel(const __grid_constant__ CUtensorMap map_k, BwdParams p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ uint64_t bar_full[kStagesA], bar_empty[kStagesA];
  __shared__ float4 sm_st[kConsumerWarps][kMaxRows];

  uint8_t* stage_base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const Item it = decode_item(p);
  const int T_b = it.T_b;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStagesA; ++s) { ptx::mbar_init(&bar_full[s], 1); ptx::mbar_init(&bar_empty[s], kConsumerWarps); }
    ptx::fence_barrier_init();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    if (lane == 0 && it.n_tiles > 0) produce_k_tiles<kStagesA>(&map_k, p, it, stage_base, bar_full, bar_empty);
    __syncwarp();
  } else {
    // Q^T fragments (B operand) in registers, as in the forward kernel
    uint32_t qb[NT][8][2];
    int lim[NT][2];
#pragma unroll
    for (int t8 = 0; t8 < NT; ++t8) {
      const int r = 8 * t8 + gid;
      const bool live = r < p.n_rows;
      const int hl = live ? r / p.w : 0, j = live ? r - hl * p.w : 0;
      const uint32_t* qrow = (const uint32_t*)((const __nv_bfloat16*)p.q_recent +
                                               ((((int64_t)it.l * p.B + it.b) * p.Hq + it.h * p.g + hl) * p.w + j) * 128);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[t8][ks][0] = live ? qrow[8 * ks + tig] : 0u;
        qb[t8][ks][1] = live ? qrow[8 * ks + tig + 4] : 0u;
      }
#pragma unroll
      for (int e = 0; e < 2; ++e) lim[t8][e] = column_limit(p, 8 * t8 + 2 * tig + e, T_b);
    }
    float m_run[NT][2], s_run[NT][2], n_run[NT][2];
#pragma unroll
    for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
      for (int e = 0; e < 2; ++e) { m_run[t8][e] = -INFINITY; s_run[t8][e] = 0.f; n_run[t8][e] = 0.f; }
    const uint32_t a_lane_off = (uint32_t)((16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * 128);
    const uint32_t x7 = (uint32_t)(lane & 7);
    const float inv_rows = inv_list_rows(p, T_b);

    for (int i = 0; i < it.n_tiles; ++i) {
      const int s = i % kStagesA;
      const int t_base = (it.tile_lo + i) * kTileT + 16 * warp;
      // the tokens' upstream weights are fetched before the wait, so that their latency hides behind it
      const int t0 = t_base + gid, t1 = t0 + 8;
      const float P0 = token_weight(p, it.b, it.gi, t0, T_b, inv_rows);
      const float P1 = token_weight(p, it.b, it.gi, t1, T_b, inv_rows);
      if (!ptx::mbar_wait_bounded(&bar_full[s], (i / kStagesA) & 1)) set_dev_status(p.dev_status, NGC_DEV_TIMEOUT);
      const uint32_t k_st = ptx::smem_u32(stage_base + s * kStageBytes);
      if (t_base < T_b) {
        float acc[NT][4];
#pragma unroll
        for (int t8 = 0; t8 < NT; ++t8) { acc[t8][0] = 0.f; acc[t8][1] = 0.f; acc[t8][2] = 0.f; acc[t8][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t chunk = (uint32_t)(2 * (ks & 3) + (lane >> 4));
          const uint32_t addr = k_st + (ks >> 2) * kBoxBytes + a_lane_off + ((chunk ^ x7) << 4);
          uint32_t a[4];
          ptx::ldmatrix_x4(addr, a[0], a[1], a[2], a[3]);
#pragma unroll
          for (int t8 = 0; t8 < NT; ++t8) ptx::mma_bf16_16816(acc[t8], a, qb[t8][ks][0], qb[t8][ks][1]);
        }
        // tokens of this slice that some row cannot see: the window itself and the tail beyond T_b
        const bool masked = t_base + 16 > T_b - p.w;
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
            const float neg = -ms * p.scale_log2;
            const float e_old = ptx::ex2_approx(fmaf(m_run[t8][e], p.scale_log2, neg));
            const float e0 = ptx::ex2_approx(fmaf(a0, p.scale_log2, neg));
            const float e1 = ptx::ex2_approx(fmaf(a1, p.scale_log2, neg));
            s_run[t8][e] = fmaf(s_run[t8][e], e_old, e0 + e1);
            n_run[t8][e] = fmaf(n_run[t8][e], e_old, fmaf(e0, P0, e1 * P1));
            m_run[t8][e] = mx;
          }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&bar_empty[s]);
    }
    // merge over the token lanes (gid), then over warps
#pragma unroll
    for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float m = m_run[t8][e] * p.scale_log2, sum = s_run[t8][e], num = n_run[t8][e];
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          const float mo = __shfl_xor_sync(0xffffffffu, m, o);
          const float so = __shfl_xor_sync(0xffffffffu, sum, o);
          const float no = __shfl_xor_sync(0xffffffffu, num, o);
          merge3(m, sum, num, mo, so, no);
        }
        if (gid == 0) sm_st[warp][8 * t8 + 2 * tig + e] = make_float4(m, sum, num, 0.f);
      }
  }
  __syncthreads();
  if (tid < kMaxRows) {
    float m = -INFINITY, sum = 0.f, num = 0.f;
    if (tid < 8 * NT) {
#pragma unroll
      for (int w2 = 0; w2 < kConsumerWarps; ++w2) merge3(m, sum, num, sm_st[w2][tid].x, sm_st[w2][tid].y, sm_st[w2][tid].z);
    }
    p.stats[((int64_t)it.strip * p.n_split + it.split) * kMaxRows + tid] = make_float4(m, sum, num, 0.f);
  }
}

// ---------------------------------------------------------------- pass 2: dK and dQ

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); }

template <int NT>
__global__ void __launch_bounds__(kThreads, 2)
score_bwd_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_gk, BwdParams p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ uint64_t bar_full[kStagesB], bar_empty[kStagesB];
  __shared__ float sm_negM[kMaxRows], sm_inv[kMaxRows], sm_c[kMaxRows];

  uint8_t* stage_base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  uint8_t* q_s = stage_base + kStagesB * kStageBytes + kStageBytes;   // [48][kQRowBytes] bf16 query rows, zero padded
  uint8_t* dz_s = q_s + kQBytes;                               // [2][64][kDzRowBytes] bf16 dz of a tile
  uint8_t* dk_s = stage_base + kStagesB * kStageBytes;         // [64][128] bf16 dK of a tile, swizzled like a K tile
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const Item it = decode_item(p);
  const int T_b = it.T_b;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStagesB; ++s) { ptx::mbar_init(&bar_full[s], 1); ptx::mbar_init(&bar_empty[s], kConsumerWarps); }
    ptx::fence_barrier_init();
  }
  if (tid < kMaxRows) {
    const float4* st = p.stats + (int64_t)it.strip * p.n_split * kMaxRows;
    float m = -INFINITY, sum = 0.f, num = 0.f;
    for (int c = 0; c < p.n_split; ++c) {
      const float4 v = st[c * kMaxRows + tid];
      merge3(m, sum, num, v.x, v.y, v.z);
    }
    const bool live = tid < p.n_rows && sum > 0.f;
    sm_negM[tid] = live ? -m : 0.f;
    sm_inv[tid] = live ? 1.f / sum : 0.f;
    sm_c[tid] = live ? num / sum : 0.f;
  }
  for (int c = tid; c < 48 * 16; c += kThreads) {              // 16-byte pieces of the query rows
    const int r = c >> 4, piece = c & 15;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < p.n_rows) {
      const int hl = r / p.w, j = r - hl * p.w;
      v = ((const uint4*)((const __nv_bfloat16*)p.q_recent +
                          ((((int64_t)it.l * p.B + it.b) * p.Hq + it.h * p.g + hl) * p.w + j) * 128))[piece];
    }
    *reinterpret_cast<uint4*>(q_s + r * kQRowBytes + piece * 16) = v;
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    if (lane == 0 && it.n_tiles > 0) produce_k_tiles<kStagesB>(&map_k, p, it, stage_base, bar_full, bar_empty);
    return;                      // the consumer warps synchronise among themselves from here on
  }

  int lim[NT][2];
  float negM[NT][2], inv[NT][2], cc[NT][2];
#pragma unroll
  for (int t8 = 0; t8 < NT; ++t8)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int c = 8 * t8 + 2 * tig + e;
      lim[t8][e] = column_limit(p, c, T_b);
      negM[t8][e] = sm_negM[c]; inv[t8][e] = sm_inv[c]; cc[t8][e] = sm_c[c];
    }
  // dQ accumulators of this warp: rows 16*mt + {gid, gid+8} x channels 32*warp + 8*n4 + {2*tig, 2*tig+1}
  float dq[3][4][4];
#pragma unroll
  for (int mt = 0; mt < 3; ++mt)
#pragma unroll
    for (int n4 = 0; n4 < 4; ++n4) { dq[mt][n4][0] = 0.f; dq[mt][n4][1] = 0.f; dq[mt][n4][2] = 0.f; dq[mt][n4][3] = 0.f; }

  const uint32_t q_u32 = ptx::smem_u32(q_s), dz_u32 = ptx::smem_u32(dz_s);
  const uint32_t x7 = (uint32_t)(lane & 7);
  const uint32_t ka_lane_off = (uint32_t)((16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * 128);   // K rows as A operand
  const uint32_t kb_lane_row = (uint32_t)((lane & 7) + 8 * ((lane >> 3) & 1));                       // K rows as B operand (tokens on k)
  const uint32_t qs_lane = (uint32_t)(((lane & 7) + 8 * (lane >> 4)) * kQRowBytes + ((lane >> 3) & 1) * 16);   // Q^T for S
  const uint32_t qk_lane = (uint32_t)(((lane & 7) + 8 * ((lane >> 3) & 1)) * kQRowBytes + (lane >> 4) * 16);   // Q for dK
  const uint32_t dz_lane = (uint32_t)(((lane & 7) + 8 * (lane >> 4)) * kDzRowBytes + ((lane >> 3) & 1) * 16);  // dZ^T for dQ
  const float inv_rows = inv_list_rows(p, T_b);
  __nv_bfloat16* gk_strip = (__nv_bfloat16*)p.grad_k + ((int64_t)(it.l * p.Hkv + it.h) * p.rows_R + p.seq_off[it.b]) * 128;

  for (int i = 0; i < it.n_tiles; ++i) {
    const int s = i % kStagesB;
    const int t_base = (it.tile_lo + i) * kTileT + 16 * warp;
    const int t0 = t_base + gid, t1 = t0 + 8;
    const float P0 = token_weight(p, it.b, it.gi, t0, T_b, inv_rows);       // fetched ahead of the wait
    const float P1 = token_weight(p, it.b, it.gi, t1, T_b, inv_rows);
    if (!ptx::mbar_wait_bounded(&bar_full[s], (i / kStagesB) & 1)) set_dev_status(p.dev_status, NGC_DEV_TIMEOUT);
    uint8_t* st = stage_base + s * kStageBytes;
    const uint32_t k_st = ptx::smem_u32(st);
    const uint32_t dz_buf = dz_u32 + (uint32_t)(i & 1) * kDzBytes;
    const int valid = T_b - t_base;                       // live tokens of this warp's slice
    if (valid < 16) {
      // rows beyond the sequence may hold anything; every warp multiplies them by dz = 0 below: zero them
      for (int x = lane; x < 16 * 16; x += 32) {
        const int r = x >> 4, c = x & 15;
        if (r >= valid) *reinterpret_cast<uint4*>(st + (c >> 3) * kBoxBytes + (16 * warp + r) * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
      }
      ptx::fence_proxy_async();      // the stage is refilled by TMA later
      __syncwarp();
    }
    // ---- S^T = K Q^T (16 tokens x 8*NT rows) ----
    float acc[NT][4];
#pragma unroll
    for (int t8 = 0; t8 < NT; ++t8) { acc[t8][0] = 0.f; acc[t8][1] = 0.f; acc[t8][2] = 0.f; acc[t8][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t chunk = (uint32_t)(2 * (ks & 3) + (lane >> 4));
      uint32_t a[4];
      ptx::ldmatrix_x4(k_st + (ks >> 2) * kBoxBytes + ka_lane_off + ((chunk ^ x7) << 4), a[0], a[1], a[2], a[3]);
#pragma unroll
      for (int t8 = 0; t8 < NT; t8 += 2) {
        uint32_t b0, b1, b2, b3;                          // Q^T fragments of row tiles t8, t8 + 1
        ptx::ldmatrix_x4(q_u32 + (uint32_t)(8 * t8) * kQRowBytes + qs_lane + ks * 32, b0, b1, b2, b3);
        ptx::mma_bf16_16816(acc[t8], a, b0, b1);
        if (t8 + 1 < NT) ptx::mma_bf16_16816(acc[t8 + 1], a, b2, b3);
      }
    }
    // ---- dz = A (P - c) / sqrt(d), packed to bf16: lo = token gid, hi = token gid + 8 ----
    uint32_t lo[6], hi[6];
#pragma unroll
    for (int t8 = 0; t8 < 6; ++t8) {
      lo[t8] = 0u; hi[t8] = 0u;
      if (t8 < NT) {
        float d0[2], d1[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float A0 = ptx::ex2_approx(fmaf(acc[t8][e], p.scale_log2, negM[t8][e])) * inv[t8][e];
          const float A1 = ptx::ex2_approx(fmaf(acc[t8][e + 2], p.scale_log2, negM[t8][e])) * inv[t8][e];
          d0[e] = t0 <= lim[t8][e] ? A0 * (P0 - cc[t8][e]) * p.inv_sqrt_d : 0.f;
          d1[e] = t1 <= lim[t8][e] ? A1 * (P1 - cc[t8][e]) * p.inv_sqrt_d : 0.f;
        }
        lo[t8] = ptx::pack_bf16x2(d0[0], d0[1]);
        hi[t8] = ptx::pack_bf16x2(d1[0], d1[1]);
      }
      // the whole tile's dz goes to shared memory for the dQ product (rows padded to 48 with zeros)
      const uint32_t off = (uint32_t)(16 * warp + gid) * kDzRowBytes + (uint32_t)(8 * t8 + 2 * tig) * 2;
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(dz_buf + off), "r"(lo[t8]) : "memory");
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(dz_buf + off + 8 * kDzRowBytes), "r"(hi[t8]) : "memory");
    }
    // ---- dK = dZ Q (16 tokens x 128 channels, 64 at a time): A operand straight from the packed dz ----
    // A tile that lies wholly inside the sequence leaves through shared memory and one TMA store per
    // 64-channel box; the sequence's last, partial tile is written row by row (rows beyond T_b stay untouched).
    const bool full_tile = (it.tile_lo + i) * kTileT + kTileT <= T_b;
    if (tid == 0) ptx::bulk_wait_read<0>();          // the previous tile's store has read the dK buffer
    consumer_bar();
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      float dk[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n) { dk[n][0] = 0.f; dk[n][1] = 0.f; dk[n][2] = 0.f; dk[n][3] = 0.f; }
#pragma unroll
      for (int kk = 0; kk < 3; ++kk) {
        if (16 * kk < 8 * NT) {
          const uint32_t a[4] = {lo[2 * kk], hi[2 * kk], lo[2 * kk + 1], hi[2 * kk + 1]};
#pragma unroll
          for (int np = 0; np < 4; ++np) {
            uint32_t r0, r1, r2, r3;
            ptx::ldmatrix_x4_trans(q_u32 + (uint32_t)(16 * kk) * kQRowBytes + qk_lane + (4 * half + np) * 32, r0, r1, r2, r3);
            ptx::mma_bf16_16816(dk[2 * np], a, r0, r1);
            ptx::mma_bf16_16816(dk[2 * np + 1], a, r2, r3);
          }
        }
      }
      if (full_tile) {
        const int ra = 16 * warp + gid, rb = ra + 8;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
          *reinterpret_cast<uint32_t*>(dk_s + half * kBoxBytes + ra * 128 + ((n ^ (ra & 7)) << 4) + 4 * tig) = ptx::pack_bf16x2(dk[n][0], dk[n][1]);
          *reinterpret_cast<uint32_t*>(dk_s + half * kBoxBytes + rb * 128 + ((n ^ (rb & 7)) << 4) + 4 * tig) = ptx::pack_bf16x2(dk[n][2], dk[n][3]);
        }
      } else {
#pragma unroll
        for (int n = 0; n < 8; ++n) {
          const int ch = 64 * half + 8 * n + 2 * tig;
          if (t0 < T_b) *reinterpret_cast<uint32_t*>(gk_strip + (int64_t)t0 * 128 + ch) = ptx::pack_bf16x2(dk[n][0], dk[n][1]);
          if (t1 < T_b) *reinterpret_cast<uint32_t*>(gk_strip + (int64_t)t1 * 128 + ch) = ptx::pack_bf16x2(dk[n][2], dk[n][3]);
        }
      }
    }
    ptx::fence_proxy_async();    // the dK tile was written through the generic proxy, the TMA store reads it
    consumer_bar();              // the tile's dz and dK are complete and dead K rows are zero
    if (tid == 0 && full_tile) {
      const int y = (int)p.seq_off[it.b] + (it.tile_lo + i) * kTileT;
      ptx::tma_store_3d(&map_gk, 0, y, it.l * p.Hkv + it.h, dk_s);
      ptx::tma_store_3d(&map_gk, 64, y, it.l * p.Hkv + it.h, dk_s + kBoxBytes);
      ptx::bulk_commit();
    }
    // ---- dQ[:, 32*warp .. +32] += dZ^T K over the 64 tokens of the tile ----
#pragma unroll
    for (int kt = 0; kt < 4; ++kt) {
      uint32_t kb[2][4];
#pragma unroll
      for (int np = 0; np < 2; ++np) {
        const uint32_t chunk = (uint32_t)(4 * (warp & 1) + 2 * np + (lane >> 4));
        ptx::ldmatrix_x4_trans(k_st + (warp >> 1) * kBoxBytes + (16 * kt + kb_lane_row) * 128 + ((chunk ^ x7) << 4),
                               kb[np][0], kb[np][1], kb[np][2], kb[np][3]);
      }
#pragma unroll
      for (int mt = 0; mt < 3; ++mt) {
        if (16 * mt < 8 * NT) {
          uint32_t a[4];
          ptx::ldmatrix_x4_trans(dz_buf + (uint32_t)(16 * kt) * kDzRowBytes + dz_lane + mt * 32, a[0], a[1], a[2], a[3]);
#pragma unroll
          for (int np = 0; np < 2; ++np) {
            ptx::mma_bf16_16816(dq[mt][2 * np], a, kb[np][0], kb[np][1]);
            ptx::mma_bf16_16816(dq[mt][2 * np + 1], a, kb[np][2], kb[np][3]);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&bar_empty[s]);
  }
  if (tid == 0) ptx::bulk_wait<0>();       // the last dK tile has left shared memory and reached global memory
  // ---- this range's dQ partial: rows x 128 channels, fp32 ----
  float* part = p.dq_part + ((int64_t)it.strip * p.n_split + it.split) * kMaxRows * 128;
#pragma unroll
  for (int mt = 0; mt < 3; ++mt)
#pragma unroll
    for (int n4 = 0; n4 < 4; ++n4) {
      const int ch = 32 * warp + 8 * n4 + 2 * tig;
      const int r0 = 16 * mt + gid, r1 = r0 + 8;
      if (r0 < p.n_rows) *reinterpret_cast<float2*>(part + r0 * 128 + ch) = make_float2(dq[mt][n4][0], dq[mt][n4][1]);
      if (r1 < p.n_rows) *reinterpret_cast<float2*>(part + r1 * 128 + ch) = make_float2(dq[mt][n4][2], dq[mt][n4][3]);
    }
}

// ---------------------------------------------------------------- pass 3: sum the ranges of a strip

__global__ void __launch_bounds__(128) score_bwd_reduce_kernel(BwdParams p) {
  const int strip = blockIdx.x / p.n_rows, r = blockIdx.x % p.n_rows;
  const int h = strip % p.Hkv, b = (strip / p.Hkv) % p.B, l = strip / (p.Hkv * p.B);
  const int hl = r / p.w, j = r - hl * p.w;
  float acc = 0.f;
  for (int s = 0; s < p.n_split; ++s) acc += p.dq_part[(((int64_t)strip * p.n_split + s) * kMaxRows + r) * 128 + threadIdx.x];
  p.grad_q[((((int64_t)l * p.B + b) * p.Hq + h * p.g + hl) * p.w + j) * 128 + threadIdx.x] = acc;
}

constexpr int kTargetCtas = 148 * 2 * 2;

int bwd_n_split(const ngc_cache* c) {
  const int64_t strips = (int64_t)c->L * c->B * c->Hkv;
  if (strips >= kTargetCtas) return 1;
  int ns = (int)((kTargetCtas + strips - 1) / strips);
  const int by_len = (c->max_len + 4 * kTileT - 1) / (4 * kTileT);
  if (ns > by_len) ns = by_len;
  if (ns > 64) ns = 64;
  return ns < 1 ? 1 : ns;
}

template <int NT>
int launch_bwd(const CUtensorMap& map_k, const CUtensorMap& map_gk, const BwdParams& p, unsigned grid, bool use_umma, cudaStream_t stream) {
  const int smem_a = kStagesA * kStageBytes + 1024;
  const int smem_b = kStagesB * kStageBytes + 1024 + kStageBytes + kQBytes + 2 * kDzBytes;
  static PerDeviceOnce attr_once;      // the shared-memory opt-in is stored per device
  const int attr_rc = attr_once.run([&] {
    cudaError_t e = cudaFuncSetAttribute(score_bwd_stats_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_a);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_bwd_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_b);
    return e;
  });
  if (attr_rc != NGC_OK) return attr_rc;
  score_bwd_stats_kernel<NT><<<grid, kThreads, smem_a, stream>>>(map_k, p);
  if (!use_umma) score_bwd_kernel<NT><<<grid, kThreads, smem_b, stream>>>(map_k, map_gk, p);
  return launch_status();
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
  CUtensorMap map_k, map_gk;
  if (!make_kv_map(&map_k, c->k, c->rows, c->L * c->Hkv, kTileT) || !make_kv_map(&map_gk, grad_k, c->rows, c->L * c->Hkv, kTileT))
    return NGC_ERR_UNSUPPORTED;
  const unsigned grid = (unsigned)items;
  const bool use_umma = getenv("NGC_BWD_LEGACY") == nullptr;
  int rc;
  switch ((p.n_rows + 7) / 8) {
    case 1: rc = launch_bwd<1>(map_k, map_gk, p, grid, use_umma, stream); break;
    case 2: rc = launch_bwd<2>(map_k, map_gk, p, grid, use_umma, stream); break;
    case 3: rc = launch_bwd<3>(map_k, map_gk, p, grid, use_umma, stream); break;
    case 4: rc = launch_bwd<4>(map_k, map_gk, p, grid, use_umma, stream); break;
    default: rc = launch_bwd<5>(map_k, map_gk, p, grid, use_umma, stream); break;
  }
  if (rc != NGC_OK) return rc;
  if (use_umma) {
    rc = launch_score_bwd_umma(p, c->k, grad_k, c->rows, c->L * c->Hkv, (int64_t)items, stream);
    if (rc != NGC_OK) return rc;
  }
  score_bwd_reduce_kernel<<<(unsigned)(c->L * c->B * c->Hkv * p.n_rows), 128, 0, stream>>>(p);
  return launch_status();
}
