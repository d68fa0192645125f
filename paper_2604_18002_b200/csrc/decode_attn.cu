// ngc_decode_attn_ragged: decode attention over the surviving cache entries
// (paper Section 4.1: generation continues conditioned on the pruned cache).
//
// Work item = (layer, sequence, KV head, token split).  Two device paths:
//
//  * bf16, d = 128, group size Hq/Hkv <= 16 (the GQA shapes): HBM-bound
//    streaming kernel.  A producer warp feeds a ring of shared-memory stages
//    with TMA tensor loads (64 tokens x 128 channels of K and of V per stage,
//    128-byte swizzle, completion on mbarriers).  Four consumer warps each own
//    16 tokens of a stage and compute the TRANSPOSED products on the tensor
//    cores (mma.sync m16n8k16): S^T = K Q^T with the tokens on M and the
//    group's heads on N = 8 (no padded head rows; the g heads that share a K/V
//    row reuse it straight from shared memory), and O^T = V^T P^T with the
//    channels on M; P^T moves from accumulator to operand layout with two
//    movmatrix transposes.  Single-pass online softmax in fp32.  Per-warp
//    partial states are merged through shared memory at the end of the item.
//  * everything else (fp32 caches, d = 64, large groups): one query head per
//    CTA, a warp per token row, fp32 FMA and warp-shuffle reductions.
//
// With n_split > 1 each item writes an unnormalised partial (m, l, o) and a
// small combine kernel merges the splits.  The new token's K/V row is handled
// inside the attention kernel: the CTA whose token range ends the strip takes
// the row from the caller's buffer (patching it into its shared-memory tile on
// the streaming path) and stores it into the cache for later steps, so no CTA
// ever reads that cache row during the call.  lens[] is bumped by a one-CTA
// kernel behind.  The kernels of a call, and consecutive calls on a stream,
// are chained by programmatic dependent launch, so each one's prologue
// overlaps its predecessor's tail.  No kernel here ever waits on another CTA.
#include <cuda.h>
#include <cuda_bf16.h>

#include "kv_map.cuh"
#include "ngc_common.cuh"
#include "ngc_plan.h"
#include "ptx.cuh"

namespace ngc {
namespace {

struct DecodeParams {
  void* k;
  void* v;
  const int64_t* seq_off;
  int32_t* lens;
  const void* q;
  const void* new_k;
  const void* new_v;
  void* out;
  float* part_o;      // [items][n_split][d]
  float2* part_ml;    // [items][n_split]  (m in log2 units, l)
  int32_t* dev_status;
  int64_t rows;
  int L, B, Hq, Hkv, d, g;
  int layer_begin, n_layers, n_split, append, out_bf16;
  float scale_log2;   // scale * log2(e)
  // paged layout (page_table != null): rows of a plane = B * pages_cap * page, seq_off unused
  const int32_t* page_table;   // [B][G][pages_cap]
  int page, pages_cap, lists, G;
  int lens_lists;              // 0: lens[B]; else lens[B][G'] of that lists mode
};

// Visible length of sequence b for this call; -1 if the appended row does not fit.
__device__ __forceinline__ int64_t seq_capacity(const DecodeParams& p, int b) {
  return p.page_table ? (int64_t)p.pages_cap * p.page : p.seq_off[b + 1] - p.seq_off[b];
}
// Visible length of strip (b, l, h) in this call; -1 if the appended row does not fit.
__device__ __forceinline__ int visible_len(const DecodeParams& p, int b, int l, int h) {
  const int len = p.lens[len_index(p.lens_lists, p.L, p.Hkv, b, l, h)];
  if (!p.append) return len;
  return (len + 1 > seq_capacity(p, b)) ? -1 : len + 1;
}

// ---------------------------------------------------------------- lens bump

__global__ void bump_lens_kernel(DecodeParams p) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();          // every CTA of the attention (and combine) kernel has read lens
  const int per_seq = lists_G(p.lens_lists, p.L, p.Hkv);      // length entries per sequence
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= p.B * per_seq) return;
  const int len = p.lens[idx];
  if (len + 1 <= seq_capacity(p, idx / per_seq)) p.lens[idx] = len + 1;
}

// ---------------------------------------------------------------- output helpers

__device__ __forceinline__ void store_out(const DecodeParams& p, int64_t idx, float v) {
  if (p.out_bf16) ((__nv_bfloat16*)p.out)[idx] = __float2bfloat16(v);
  else ((float*)p.out)[idx] = v;
}

// ---------------------------------------------------------------- generic path

template <typename T> struct RowLoad;
template <> struct RowLoad<float> {
  template <int VPL> static __device__ __forceinline__ void load(const float* row, int lane, float (&x)[VPL]) {
    if constexpr (VPL == 2) {
      const float2 t = ((const float2*)row)[lane];
      x[0] = t.x; x[1] = t.y;
    } else {
      const float4 t = ((const float4*)row)[lane];
      x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
    }
  }
};
template <> struct RowLoad<__nv_bfloat16> {
  template <int VPL> static __device__ __forceinline__ void load(const __nv_bfloat16* row, int lane, float (&x)[VPL]) {
    if constexpr (VPL == 2) {
      const __nv_bfloat162 t = ((const __nv_bfloat162*)row)[lane];
      x[0] = __low2float(t); x[1] = __high2float(t);
    } else {
      const uint2 t = ((const uint2*)row)[lane];
      const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
      const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
      x[0] = __low2float(a); x[1] = __high2float(a); x[2] = __low2float(c); x[3] = __high2float(c);
    }
  }
};

constexpr int kGenWarps = 4;
constexpr int kGenChunk = 64;   // split granularity in tokens (same as the streaming path)

template <typename T, int D>
__global__ void __launch_bounds__(kGenWarps * 32) decode_generic_kernel(DecodeParams p) {
  constexpr int VPL = D / 32;
  __shared__ float sm_m[kGenWarps], sm_l[kGenWarps];
  __shared__ float sm_acc[kGenWarps][D];

  int item = blockIdx.x;
  const int split = item % p.n_split; item /= p.n_split;
  const int hq = item % p.Hq;
  const int b = (item / p.Hq) % p.B;
  const int lr = item / (p.Hq * p.B);
  const int l = p.layer_begin + lr;
  const int h = hq / p.g;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  int len = visible_len(p, b, l, h);
  if (len < 0) {
    if (tid == 0) set_dev_status(p.dev_status, NGC_DEV_STRIP_FULL);
    len = 0;
  }
  const int t_new = (p.append && len > 0) ? len - 1 : -1;      // position of the appended row
  const int nt = (len + kGenChunk - 1) / kGenChunk;
  const int tps = (nt + p.n_split - 1) / p.n_split;
  const int t_begin = min(len, split * tps * kGenChunk);
  const int t_end = min(len, (split + 1) * tps * kGenChunk);

  const int64_t qo = (((int64_t)l * p.B + b) * p.Hq + hq) * D;
  float qv[VPL];
  RowLoad<T>::template load<VPL>((const T*)p.q + qo, lane, qv);
  T* kbase = (T*)p.k + ((int64_t)(l * p.Hkv + h) * p.rows + p.seq_off[b]) * D;
  T* vbase = (T*)p.v + ((int64_t)(l * p.Hkv + h) * p.rows + p.seq_off[b]) * D;
  const T* knew = (const T*)p.new_k + (((int64_t)l * p.B + b) * p.Hkv + h) * D;
  const T* vnew = (const T*)p.new_v + (((int64_t)l * p.B + b) * p.Hkv + h) * D;

  float m = -INFINITY, lsum = 0.f, acc[VPL];
#pragma unroll
  for (int i = 0; i < VPL; ++i) acc[i] = 0.f;
  for (int t = t_begin + warp; t < t_end; t += kGenWarps) {
    float kx[VPL], vx[VPL];
    // the appended row is taken from the caller's buffer: its cache row is written during this launch
    RowLoad<T>::template load<VPL>(t == t_new ? knew : kbase + (int64_t)t * D, lane, kx);
    RowLoad<T>::template load<VPL>(t == t_new ? vnew : vbase + (int64_t)t * D, lane, vx);
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < VPL; ++i) dot = fmaf(qv[i], kx[i], dot);
    dot = warp_sum(dot);
    const float z = dot * p.scale_log2;
    const float m_new = fmaxf(m, z);
    const float alpha = exp2f(m - m_new);
    const float pz = exp2f(z - m_new);
    lsum = lsum * alpha + pz;
#pragma unroll
    for (int i = 0; i < VPL; ++i) acc[i] = fmaf(pz, vx[i], acc[i] * alpha);
    m = m_new;
  }
  // one CTA per KV head stores the appended row for the following steps
  if (t_new >= t_begin && t_new < t_end && hq == h * p.g && warp < 2) {
    const T* src = warp ? vnew : knew;
    T* dst = (warp ? vbase : kbase) + (int64_t)t_new * D;
    if (NGC_IN_BOUNDS(p.dev_status, t_new < p.seq_off[b + 1] - p.seq_off[b])) {
#pragma unroll
      for (int i = 0; i < VPL; ++i) dst[lane * VPL + i] = src[lane * VPL + i];
    }
  }
  if (lane == 0) { sm_m[warp] = m; sm_l[warp] = lsum; }
#pragma unroll
  for (int i = 0; i < VPL; ++i) sm_acc[warp][lane * VPL + i] = acc[i];
  __syncthreads();
  if (tid < D) {
    float mg = sm_m[0];
#pragma unroll
    for (int w = 1; w < kGenWarps; ++w) mg = fmaxf(mg, sm_m[w]);
    float o = 0.f, ls = 0.f;
#pragma unroll
    for (int w = 0; w < kGenWarps; ++w) {
      const float f = sm_m[w] == -INFINITY ? 0.f : exp2f(sm_m[w] - mg);
      o = fmaf(sm_acc[w][tid], f, o);
      ls = fmaf(sm_l[w], f, ls);
    }
    const int64_t it = ((int64_t)lr * p.B + b) * p.Hq + hq;
    if (p.n_split == 1) {
      store_out(p, qo + tid, ls > 0.f ? o / ls : 0.f);
    } else {
      p.part_o[(it * p.n_split + split) * D + tid] = o;
      if (tid == 0) p.part_ml[it * p.n_split + split] = make_float2(mg, ls);
    }
  }
}

// ---------------------------------------------------------------- split combine

__global__ void combine_kernel(DecodeParams p) {
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  const int64_t it = blockIdx.x;               // (lr, b, hq)
  const int c = threadIdx.x;                   // channel
  const int lr = (int)(it / ((int64_t)p.B * p.Hq));
  const int64_t rest = it - (int64_t)lr * p.B * p.Hq;
  const int64_t qo = (((int64_t)(p.layer_begin + lr) * p.B) * p.Hq + rest) * p.d;
  float mg = -INFINITY;
  for (int s = 0; s < p.n_split; ++s) mg = fmaxf(mg, p.part_ml[it * p.n_split + s].x);
  float o = 0.f, ls = 0.f;
  for (int s = 0; s < p.n_split; ++s) {
    const float2 ml = p.part_ml[it * p.n_split + s];
    const float f = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mg);
    o = fmaf(p.part_o[(it * p.n_split + s) * p.d + c], f, o);
    ls = fmaf(ml.y, f, ls);
  }
  store_out(p, qo + c, ls > 0.f ? o / ls : 0.f);
}

// ---------------------------------------------------------------- streaming bf16 path

constexpr int kTileT = 64;                    // tokens per stage
constexpr int kConsumerWarps = 4;
constexpr int kStreamThreads = (kConsumerWarps + 1) * 32;
constexpr int kBoxBytes = kTileT * 128;       // one 64 x 64 bf16 box
constexpr int kTileBytes = 2 * kBoxBytes;     // K (or V) tile: two boxes (channels 0-63, 64-127)
constexpr int kStageBytes = 2 * kTileBytes;   // K + V
constexpr int kStages1 = 2, kMinCtas1 = 3;    // groups of <= 8 heads: 128 registers, 2-stage ring, 3 CTAs per SM
constexpr int kStages2 = 3, kMinCtas2 = 2;    // groups of 9..16 heads: two head tiles, 3-stage ring, 2 CTAs per SM
constexpr int kORowStride = 132;              // floats; merge buffer row stride (bank spread)

// Tensor maps of a launch: K and V with the full-tile box (64 rows, or one page) and with a
// 16-row box for the last, partly filled tile of a strip.
struct KvMaps { CUtensorMap k, v, k16, v16; };

// Issues the TMA loads of 64-token tile `tile` of a strip into stage `st` (K rows at 0, V rows at
// kTileBytes; channels 64-127 one box further).  A full tile is fetched whole (page by page on a
// paged cache).  The strip's last tile is fetched in 16-row boxes, only as many as hold live
// tokens: with caches of a few hundred tokens a whole tile for the tail would be several per cent
// of the traffic.  Sets the stage's expected byte count itself.
__device__ __forceinline__ void issue_tile(const DecodeParams& p, const KvMaps& m, const int32_t* table, int row0, int b,
                                           int plane, int tile, int len, uint8_t* st, uint64_t* bar) {
  const int t0 = tile * kTileT;
  if (t0 + kTileT <= len) {
    ptx::mbar_expect_tx(bar, kStageBytes);
    const int n_sub = table ? kTileT / p.page : 1;          // pages per 64-token tile
    const int sub_bytes = (kTileT / n_sub) * 128;
    for (int sb = 0; sb < n_sub; ++sb) {
      const int y = table ? (b * p.pages_cap + table[tile * n_sub + sb]) * p.page : row0 + t0;
      uint8_t* dst = st + sb * sub_bytes;
      // a full tile lies inside the plane (an out-of-range TMA box would read zeros, not fault: a wrong answer)
      if (!NGC_IN_BOUNDS(p.dev_status, y >= 0 && (int64_t)y + kTileT / n_sub <= p.rows &&
                                           (!table || (tile * n_sub + sb < p.pages_cap && table[tile * n_sub + sb] >= 0 &&
                                                       table[tile * n_sub + sb] < p.pages_cap)))) {
        // keep the byte count of the stage right so that the consumers are released: fetch row 0 instead
        ptx::tma_load_3d(dst, &m.k, 0, 0, plane, bar);
        ptx::tma_load_3d(dst + kBoxBytes, &m.k, 64, 0, plane, bar);
        ptx::tma_load_3d(dst + kTileBytes, &m.v, 0, 0, plane, bar);
        ptx::tma_load_3d(dst + kTileBytes + kBoxBytes, &m.v, 64, 0, plane, bar);
        continue;
      }
      ptx::tma_load_3d(dst, &m.k, 0, y, plane, bar);
      ptx::tma_load_3d(dst + kBoxBytes, &m.k, 64, y, plane, bar);
      ptx::tma_load_3d(dst + kTileBytes, &m.v, 0, y, plane, bar);
      ptx::tma_load_3d(dst + kTileBytes + kBoxBytes, &m.v, 64, y, plane, bar);
    }
  } else {
    const int n16 = (len - t0 + 15) >> 4;                   // 1..4 groups of 16 rows
    ptx::mbar_expect_tx(bar, (uint32_t)n16 * 4 * 16 * 128);
    for (int r = 0; r < n16; ++r) {
      const int t = t0 + 16 * r;
      int y = table ? (b * p.pages_cap + table[t / p.page]) * p.page + t % p.page : row0 + t;
      uint8_t* dst = st + r * 16 * 128;
      // the first row of every 16-row box holds a live token, hence lies inside the plane
      if (!NGC_IN_BOUNDS(p.dev_status, y >= 0 && y < p.rows && (!table || t / p.page < p.pages_cap))) y = 0;
      ptx::tma_load_3d(dst, &m.k16, 0, y, plane, bar);
      ptx::tma_load_3d(dst + kBoxBytes, &m.k16, 64, y, plane, bar);
      ptx::tma_load_3d(dst + kTileBytes, &m.v16, 0, y, plane, bar);
      ptx::tma_load_3d(dst + kTileBytes + kBoxBytes, &m.v16, 64, y, plane, bar);
    }
  }
}

// The streaming kernel.  NH = 8-head tiles of the group (1: groups of at most 8 heads, every GQA shape of
// the paper's model family; 2: groups of 9..16 heads).
template <int NH, int kNStages, int kMinCtas>
__global__ void __launch_bounds__(kStreamThreads, kMinCtas)
decode_stream_t_kernel(const __grid_constant__ KvMaps maps, DecodeParams p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ uint64_t bar_full[kNStages], bar_empty[kNStages];
  __shared__ float sm_m[kConsumerWarps][8 * NH], sm_l[kConsumerWarps][8 * NH];

  uint8_t* stage_base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;

  int item = blockIdx.x;
  const int split = item % p.n_split; item /= p.n_split;
  const int h = item % p.Hkv;
  const int b = (item / p.Hkv) % p.B;
  const int lr = item / (p.Hkv * p.B);
  const int l = p.layer_begin + lr;
  const int g = p.g;
  const int32_t* table = p.page_table
      ? p.page_table + ((int64_t)b * p.G + list_of(p.lists, l, h, p.Hkv)) * p.pages_cap : nullptr;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kNStages; ++s) { ptx::mbar_init(&bar_full[s], 1); ptx::mbar_init(&bar_empty[s], kConsumerWarps); }
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&maps.k);
    ptx::prefetch_tensormap(&maps.v);
  }
  ptx::grid_dep_wait();           // lens and the cache rows of earlier calls are final from here on
  ptx::grid_dep_launch();

  int len = visible_len(p, b, l, h);
  if (len < 0) {
    if (tid == 0) set_dev_status(p.dev_status, NGC_DEV_STRIP_FULL);
    len = 0;
  }
  const int t_new = (p.append && len > 0) ? len - 1 : -1;      // position of the appended row
  const int nt = (len + kTileT - 1) / kTileT;
  const int tps = (nt + p.n_split - 1) / p.n_split;
  const int tile_lo = min(nt, split * tps);
  const int tile_hi = min(nt, tile_lo + tps);
  const int n_tiles = tile_hi - tile_lo;
  __syncthreads();

  // O^T accumulators: o_acc[t][mt] = channels 16*mt + {gid, gid+8} x heads 8*t + {2*tig, 2*tig+1}
  float o_acc[NH][8][4];
  float m_run[NH][2], l_run[NH][2];             // running max / sum of heads 8*t + 2*tig, + 1 (log2 domain)
#pragma unroll
  for (int t = 0; t < NH; ++t) {
    m_run[t][0] = -INFINITY; m_run[t][1] = -INFINITY; l_run[t][0] = 0.f; l_run[t][1] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) { o_acc[t][i][0] = 0.f; o_acc[t][i][1] = 0.f; o_acc[t][i][2] = 0.f; o_acc[t][i][3] = 0.f; }
  }

  if (warp == kConsumerWarps) {
    // ------------------------------------------------ producer
    if (lane == 0 && n_tiles > 0) {
      const int plane = l * p.Hkv + h;
      const int row0 = table ? 0 : (int)p.seq_off[b];
      for (int it = 0; it < n_tiles; ++it) {
        const int s = it % kNStages;
        if (it >= kNStages) {
          if (!ptx::mbar_wait_bounded(&bar_empty[s], ((it / kNStages) - 1) & 1)) set_dev_status(p.dev_status, NGC_DEV_TIMEOUT);
        }
        issue_tile(p, maps, table, row0, b, plane, tile_lo + it, len, stage_base + s * kStageBytes, &bar_full[s]);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ consumers
    // Transposed products: S^T = K Q^T (16 tokens x 8 heads) and O^T = V^T P^T (128 channels x 8
    // heads) per tile of 8 heads, so the heads of the group sit on the N = 8 axis of the MMA.
    // Q^T fragments (B operand, column n = head gid): zero beyond g.
    uint32_t qb[NH][8][2];
#pragma unroll
    for (int t = 0; t < NH; ++t) {
      const uint32_t* q0 = (const uint32_t*)((const __nv_bfloat16*)p.q + (((int64_t)l * p.B + b) * p.Hq + h * g + 8 * t + gid) * 128);
      const bool live = 8 * t + gid < g;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[t][ks][0] = live ? q0[8 * ks + tig] : 0u;
        qb[t][ks][1] = live ? q0[8 * ks + tig + 4] : 0u;
      }
    }
    // lane-dependent parts of the swizzled shared-memory addresses
    const uint32_t k_lane_off = (uint32_t)((16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * 128);   // A operand, K rows
    const uint32_t v_lane_off = (uint32_t)((16 * warp + (lane & 7) + 8 * (lane >> 4)) * 128);         // A operand, V^T
    const uint32_t x7 = (uint32_t)(lane & 7);

    const bool own_new = t_new >= 0 && tile_hi == nt && n_tiles > 0 && ((t_new % kTileT) >> 4) == warp;
    uint4 piece = make_uint4(0, 0, 0, 0);
    if (own_new)
      piece = ((const uint4*)((lane >> 4) ? p.new_v : p.new_k))[(((int64_t)l * p.B + b) * p.Hkv + h) * 16 + (lane & 15)];

    for (int it = 0; it < n_tiles; ++it) {
      const int s = it % kNStages;
      if (!ptx::mbar_wait_bounded(&bar_full[s], (it / kNStages) & 1)) set_dev_status(p.dev_status, NGC_DEV_TIMEOUT);
      uint8_t* st = stage_base + s * kStageBytes;
      const uint32_t k_st = ptx::smem_u32(st);
      const uint32_t v_st = k_st + kTileBytes;
      const int tile_t0 = (tile_lo + it) * kTileT;
      const int valid = len - tile_t0 - 16 * warp;      // live tokens in this warp's slice (may exceed 16)

      if (own_new && it == n_tiles - 1) {
        // the appended row: from the caller's buffer into the tile and into the cache
        const int isv = lane >> 4, c = lane & 15, r = t_new - tile_t0;
        uint8_t* dst = st + isv * kTileBytes + (c >> 3) * kBoxBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);
        *reinterpret_cast<uint4*>(dst) = piece;
        const int64_t row = table ? ((int64_t)b * p.pages_cap + table[t_new / p.page]) * p.page + t_new % p.page
                                  : p.seq_off[b] + t_new;
        if (NGC_IN_BOUNDS(p.dev_status, row >= 0 && row < p.rows && t_new < seq_capacity(p, b)))
          ((uint4*)(isv ? p.v : p.k))[((int64_t)(l * p.Hkv + h) * p.rows + row) * 16 + c] = piece;
        ptx::fence_proxy_async();
        __syncwarp();
      }
      if (valid > 0) {
        if (valid < 16) {
          // dead V rows may hold anything (NaN x 0 would poison the sum): zero them
          for (int i = lane; i < 16 * 16; i += 32) {
            const int r = i >> 4, c = i & 15;
            if (r >= valid) {
              uint8_t* rowp = st + kTileBytes + (c >> 3) * kBoxBytes + (16 * warp + r) * 128 + (c & 7) * 16;
              *reinterpret_cast<uint4*>(rowp) = make_uint4(0, 0, 0, 0);
            }
          }
          __syncwarp();
        }
        // ---- S^T = K Q^T: 16 tokens x 8 heads ----
        float sc[NH][4];                        // (tok gid, head 2tig), (gid, 2tig+1), (gid+8, 2tig), (gid+8, 2tig+1)
#pragma unroll
        for (int t = 0; t < NH; ++t) { sc[t][0] = 0.f; sc[t][1] = 0.f; sc[t][2] = 0.f; sc[t][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t chunk = (uint32_t)(2 * (ks & 3) + (lane >> 4));
          const uint32_t addr = k_st + (ks >> 2) * kBoxBytes + k_lane_off + ((chunk ^ x7) << 4);
          uint32_t a[4];
          ptx::ldmatrix_x4(addr, a[0], a[1], a[2], a[3]);
#pragma unroll
          for (int t = 0; t < NH; ++t) ptx::mma_bf16_16816(sc[t], a, qb[t][ks][0], qb[t][ks][1]);
        }
        // ---- online softmax per head (log2 domain) ----
        uint32_t pb[NH][2];
        bool changed = false;
        float alpha[NH][2];
#pragma unroll
        for (int t = 0; t < NH; ++t) {
          sc[t][0] = gid < valid ? sc[t][0] * p.scale_log2 : -INFINITY;
          sc[t][1] = gid < valid ? sc[t][1] * p.scale_log2 : -INFINITY;
          sc[t][2] = gid + 8 < valid ? sc[t][2] * p.scale_log2 : -INFINITY;
          sc[t][3] = gid + 8 < valid ? sc[t][3] * p.scale_log2 : -INFINITY;
          float mx[2] = {fmaxf(sc[t][0], sc[t][2]), fmaxf(sc[t][1], sc[t][3])};
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 4));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 8));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 16));
            const float m_new = fmaxf(m_run[t][r], mx[r]);          // finite: token 0 of the slice is live
            alpha[t][r] = ptx::ex2_approx(m_run[t][r] - m_new);
            changed = changed || m_new != m_run[t][r];
            m_run[t][r] = m_new;
          }
        }
        if (__any_sync(0xffffffffu, changed)) {
#pragma unroll
          for (int t = 0; t < NH; ++t) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              o_acc[t][i][0] *= alpha[t][0]; o_acc[t][i][1] *= alpha[t][1];
              o_acc[t][i][2] *= alpha[t][0]; o_acc[t][i][3] *= alpha[t][1];
            }
            l_run[t][0] *= alpha[t][0];
            l_run[t][1] *= alpha[t][1];
          }
        }
#pragma unroll
        for (int t = 0; t < NH; ++t) {
          float pr[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            pr[e] = ptx::ex2_approx(sc[t][e] - m_run[t][e & 1]);
            l_run[t][e & 1] += pr[e];
          }
          // P^T as B operand (k = token, n = head): transpose the two 8 x 8 (token x head) blocks
          pb[t][0] = ptx::movmatrix_trans(ptx::pack_bf16x2(pr[0], pr[1]));
          pb[t][1] = ptx::movmatrix_trans(ptx::pack_bf16x2(pr[2], pr[3]));
        }
        // ---- O^T += V^T P^T (128 channels x 8 heads per tile of heads) ----
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          const uint32_t chunk = (uint32_t)(2 * (mt & 3) + ((lane >> 3) & 1));
          const uint32_t addr = v_st + (mt >> 2) * kBoxBytes + v_lane_off + ((chunk ^ x7) << 4);
          uint32_t a[4];
          ptx::ldmatrix_x4_trans(addr, a[0], a[1], a[2], a[3]);
#pragma unroll
          for (int t = 0; t < NH; ++t) ptx::mma_bf16_16816(o_acc[t][mt], a, pb[t][0], pb[t][1]);
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&bar_empty[s]);
    }
    // row sums over the tokens of the slice (spread over gid), then publish this warp's state
#pragma unroll
    for (int t = 0; t < NH; ++t) {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 4);
        l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 8);
        l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 16);
      }
      if (gid == 0) {
        sm_m[warp][8 * t + 2 * tig] = m_run[t][0]; sm_m[warp][8 * t + 2 * tig + 1] = m_run[t][1];
        sm_l[warp][8 * t + 2 * tig] = l_run[t][0]; sm_l[warp][8 * t + 2 * tig + 1] = l_run[t][1];
      }
    }
  }
  __syncthreads();   // every stage has been consumed; the ring is free for the merge buffer

  float* obuf = reinterpret_cast<float*>(stage_base);      // [warp][8 * NH heads][kORowStride]
  if (warp < kConsumerWarps) {
#pragma unroll
    for (int t = 0; t < NH; ++t) {
      float f[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int row = 8 * t + 2 * tig + r;
        float mg = sm_m[0][row];
#pragma unroll
        for (int w = 1; w < kConsumerWarps; ++w) mg = fmaxf(mg, sm_m[w][row]);
        f[r] = m_run[t][r] == -INFINITY ? 0.f : ptx::ex2_approx(m_run[t][r] - mg);
      }
      float* ob = obuf + (warp * 8 * NH + 8 * t) * kORowStride;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        ob[(2 * tig) * kORowStride + 16 * i + gid] = o_acc[t][i][0] * f[0];
        ob[(2 * tig + 1) * kORowStride + 16 * i + gid] = o_acc[t][i][1] * f[1];
        ob[(2 * tig) * kORowStride + 16 * i + gid + 8] = o_acc[t][i][2] * f[0];
        ob[(2 * tig + 1) * kORowStride + 16 * i + gid + 8] = o_acc[t][i][3] * f[1];
      }
    }
  }
  __syncthreads();
  if (tid < 128) {
    const int c = tid;
    for (int row = 0; row < g; ++row) {
      float mg = sm_m[0][row];
#pragma unroll
      for (int w = 1; w < kConsumerWarps; ++w) mg = fmaxf(mg, sm_m[w][row]);
      float o = 0.f, ls = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        o += obuf[(w * 8 * NH + row) * kORowStride + c];
        const float mw = sm_m[w][row];
        ls += mw == -INFINITY ? 0.f : sm_l[w][row] * ptx::ex2_approx(mw - mg);
      }
      const int hq = h * g + row;
      if (p.n_split == 1) {
        store_out(p, (((int64_t)l * p.B + b) * p.Hq + hq) * 128 + c, ls > 0.f ? o / ls : 0.f);
      } else {
        const int64_t pit = (((int64_t)lr * p.B + b) * p.Hq + hq) * p.n_split + split;
        if (NGC_IN_BOUNDS(p.dev_status, pit >= 0 && pit < (int64_t)p.n_layers * p.B * p.Hq * p.n_split)) {
          p.part_o[pit * 128 + c] = o;
          if (c == 0) p.part_ml[pit] = make_float2(mg, ls);
        }
      }
    }
  }
}

// ---------------------------------------------------------------- host side

constexpr int kTargetCtas = 148 * 2 * 2;    // two waves of two CTAs per SM
constexpr int kTargetCtasT = 148 * 3 * 2;   // ... of three per SM (the kernel for groups of <= 8 heads)

}  // namespace

int decode_n_split(const ngc_cache* c, int layers) {
  const int64_t strips = (int64_t)layers * c->B * c->Hkv;
  const bool t_kernel = c->dtype == NGC_BF16 && c->d == 128 && c->Hq / c->Hkv <= 8;
  const int target = t_kernel ? kTargetCtasT : kTargetCtas;
  if (strips >= target) return 1;
  int ns = (int)((target + strips - 1) / strips);
  const int by_len = (c->max_len + 1 + 4 * kTileT - 1) / (4 * kTileT);   // at least 4 tiles per split
  if (ns > by_len) ns = by_len;
  if (ns > 64) ns = 64;
  return ns < 1 ? 1 : ns;
}

// Scratch of ONE call over `n_layers` layers: the split partials, o [items][d] fp32 then (m, l) [items]
// (0 when the call does not split).  *ml_offset (if given) gets the byte offset of the (m, l) array.
size_t decode_call_scratch_bytes(const ngc_cache* c, int n_layers, size_t* ml_offset) {
  const int ns = decode_n_split(c, n_layers);
  if (ml_offset) *ml_offset = 0;
  if (ns <= 1) return 0;
  const size_t items = (size_t)n_layers * c->B * c->Hq * ns;
  const size_t o_bytes = align256(items * c->d * 4);
  if (ml_offset) *ml_offset = o_bytes;
  return o_bytes + align256(items * 8);
}

// Workspace that serves a call over any layer range of up to `layers` layers.
size_t decode_workspace_bytes(const ngc_cache* c, int layers) {
  size_t worst = 0;
  for (int n = 1; n <= layers; ++n) {
    const size_t bytes = decode_call_scratch_bytes(c, n, nullptr);
    if (bytes > worst) worst = bytes;
  }
  return worst;
}

}  // namespace ngc

namespace ngc {
namespace {

int decode_impl(ngc_cache* c, const PagedView& pv, const void* q, const void* new_k, const void* new_v,
                int layer_begin, int layer_end, float scale, void* out, int out_dtype,
                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t stream) {
  if (!q || !out || layer_begin < 0 || layer_end > c->L || layer_begin >= layer_end)
    return NGC_ERR_INVALID_ARG;
  if ((new_k == nullptr) != (new_v == nullptr)) return NGC_ERR_INVALID_ARG;
  if ((((uintptr_t)q | (uintptr_t)new_k | (uintptr_t)new_v | (uintptr_t)out | (uintptr_t)c->k | (uintptr_t)c->v) & 15) != 0)
    return NGC_ERR_INVALID_ARG;      // rows are moved as 16-byte vectors
  if (out_dtype != NGC_F32 && !(out_dtype == NGC_BF16 && c->dtype == NGC_BF16)) return NGC_ERR_INVALID_ARG;
  if (c->rows == 0) return NGC_OK;

  DecodeParams p;
  p.k = c->k; p.v = c->v; p.seq_off = c->seq_off; p.lens = c->lens;
  p.q = q; p.new_k = new_k; p.new_v = new_v; p.out = out;
  p.dev_status = dev_status; p.rows = c->rows;
  p.L = c->L; p.B = c->B; p.Hq = c->Hq; p.Hkv = c->Hkv; p.d = c->d; p.g = c->Hq / c->Hkv;
  p.layer_begin = layer_begin; p.n_layers = layer_end - layer_begin;
  p.append = new_k != nullptr; p.out_bf16 = out_dtype == NGC_BF16;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.n_split = decode_n_split(c, p.n_layers);
  p.part_o = nullptr; p.part_ml = nullptr;
  p.page_table = pv.table; p.page = pv.page; p.pages_cap = pv.pages_cap; p.lists = pv.lists;
  p.lens_lists = c->lens_lists;
  p.G = lists_G(pv.lists, c->L, c->Hkv);
  if (p.n_split > 1) {
    size_t ml_offset = 0;
    const size_t need = decode_call_scratch_bytes(c, p.n_layers, &ml_offset);
    if (!ws || ws_bytes < need || ((uintptr_t)ws & 255)) return NGC_ERR_WORKSPACE;
    p.part_o = (float*)ws;
    p.part_ml = (float2*)((char*)ws + ml_offset);
  }

  const bool stream_path = c->dtype == NGC_BF16 && c->d == 128 && p.g <= 16 && c->rows < 0x7fffffffLL;
  if (pv.table && !stream_path) return NGC_ERR_UNSUPPORTED;          // paged caches: bf16, d = 128, groups of up to 16 heads
  if (stream_path) {
    KvMaps maps;
    const int box_rows = pv.table ? pv.page : kTileT;                 // a page is fetched as its own box
    const int planes = c->L * c->Hkv;
    if (!make_kv_map(&maps.k, c->k, c->rows, planes, box_rows) || !make_kv_map(&maps.v, c->v, c->rows, planes, box_rows) ||
        !make_kv_map(&maps.k16, c->k, c->rows, planes, 16) || !make_kv_map(&maps.v16, c->v, c->rows, planes, 16))
      return NGC_ERR_UNSUPPORTED;
    const int64_t items = (int64_t)p.n_layers * c->B * c->Hkv * p.n_split;
    if (items > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
    // the opt-in to more than 48 KB of dynamic shared memory is stored per device
    static PerDeviceOnce attr_once;
    const int attr_rc = attr_once.run([] {
      cudaError_t e = cudaFuncSetAttribute(decode_stream_t_kernel<1, kStages1, kMinCtas1>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, kStages1 * kStageBytes + 1024);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(decode_stream_t_kernel<2, kStages2, kMinCtas2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kStages2 * kStageBytes + 1024);
      return e;
    });
    if (attr_rc != NGC_OK) return attr_rc;
    if (p.g <= 8)
      NGC_CUDA_TRY(launch_pdl(decode_stream_t_kernel<1, kStages1, kMinCtas1>, dim3((unsigned)items), dim3(kStreamThreads),
                              kStages1 * kStageBytes + 1024, stream, maps, p));
    else
      NGC_CUDA_TRY(launch_pdl(decode_stream_t_kernel<2, kStages2, kMinCtas2>, dim3((unsigned)items), dim3(kStreamThreads),
                              kStages2 * kStageBytes + 1024, stream, maps, p));
  } else {
    const int64_t items = (int64_t)p.n_layers * c->B * c->Hq * p.n_split;
    if (items > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)items;
    const dim3 blk(kGenWarps * 32);
    if (c->dtype == NGC_F32 && c->d == 64) NGC_CUDA_TRY(launch_pdl(decode_generic_kernel<float, 64>, dim3(grid), blk, 0, stream, p));
    else if (c->dtype == NGC_F32) NGC_CUDA_TRY(launch_pdl(decode_generic_kernel<float, 128>, dim3(grid), blk, 0, stream, p));
    else if (c->d == 64) NGC_CUDA_TRY(launch_pdl(decode_generic_kernel<__nv_bfloat16, 64>, dim3(grid), blk, 0, stream, p));
    else NGC_CUDA_TRY(launch_pdl(decode_generic_kernel<__nv_bfloat16, 128>, dim3(grid), blk, 0, stream, p));
  }
  if (p.n_split > 1)
    NGC_CUDA_TRY(launch_pdl(combine_kernel, dim3((unsigned)(p.n_layers * c->B * c->Hq)), dim3(c->d), 0, stream, p));
  if (p.append && layer_end == c->L)
    NGC_CUDA_TRY(launch_pdl(bump_lens_kernel, dim3((c->B * lists_G(c->lens_lists, c->L, c->Hkv) + 255) / 256), dim3(256), 0, stream, p));
  return NGC_OK;
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_decode_attn_ragged(ngc_cache* c, const void* q, const void* new_k, const void* new_v,
                                      int layer_begin, int layer_end, float scale,
                                      void* out, int out_dtype,
                                      void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_decode_attn_ragged");
  using namespace ngc;
  if (!valid_cache(c)) return NGC_ERR_INVALID_ARG;
  const PagedView none = {nullptr, 0, 0, NGC_LISTS_SHARED};
  return decode_impl(c, none, q, new_k, new_v, layer_begin, layer_end, scale, out, out_dtype, ws, ws_bytes, dev_status,
                     (cudaStream_t)stream);
}

extern "C" int ngc_decode_attn_paged(ngc_paged_cache* pc, const void* q, const void* new_k, const void* new_v,
                                     int layer_begin, int layer_end, float scale,
                                     void* out, int out_dtype,
                                     void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_decode_attn_paged");
  using namespace ngc;
  if (!pc || !pc->k || !pc->v || !pc->page_table || !pc->lens || pc->L <= 0 || pc->B <= 0 || pc->Hq <= 0 || pc->Hkv <= 0 ||
      pc->Hq % pc->Hkv != 0 || pc->pages_cap <= 0 || (pc->page != 32 && pc->page != 64) || pc->lists < 0 || pc->lists > 2)
    return NGC_ERR_INVALID_ARG;
  if (pc->dtype != NGC_BF16 || pc->d != 128) return NGC_ERR_UNSUPPORTED;
  // the same kernels run on a descriptor whose planes are the page pools
  ngc_cache c;
  c.k = pc->k; c.v = pc->v; c.seq_off = nullptr; c.lens = pc->lens;
  c.rows = (int64_t)pc->B * pc->pages_cap * pc->page;
  c.L = pc->L; c.B = pc->B; c.Hq = pc->Hq; c.Hkv = pc->Hkv; c.d = pc->d; c.dtype = pc->dtype;
  c.max_len = pc->pages_cap * pc->page;
  c.lens_lists = pc->lens_per_list ? pc->lists : 0;
  const PagedView pv = {pc->page_table, pc->page, pc->pages_cap, pc->lists};
  return decode_impl(&c, pv, q, new_k, new_v, layer_begin, layer_end, scale, out, out_dtype, ws, ws_bytes, dev_status,
                     (cudaStream_t)stream);
}

// ---------------------------------------------------------------- allocation-free variant
//
// For callers that cannot provide device scratch (no allocator access, all
// memory owned by a host framework's pool, or no tolerance for cudaMalloc's
// device-wide synchronisation): the split partials go to an array that is
// part of the library image.  In host code the array's name is only a
// host-side stand-in, never a device address; the address is looked up once
// per device with cudaGetSymbolAddress while that device is current.
namespace ngc {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[NGC_STATIC_SCRATCH_BYTES];

PerDeviceOnce g_static_scratch_once;
void* g_static_scratch_addr[kMaxDevices] = {nullptr};

}  // namespace
}  // namespace ngc

extern "C" int ngc_decode_attn_ragged_static(ngc_cache* c, const void* q, const void* new_k, const void* new_v,
                                             int layer_begin, int layer_end, float scale,
                                             void* out, int out_dtype, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_decode_attn_ragged_static");
  using namespace ngc;
  if (!valid_cache(c) || layer_begin < 0 || layer_end > c->L || layer_begin >= layer_end) return NGC_ERR_INVALID_ARG;
  if (decode_call_scratch_bytes(c, layer_end - layer_begin, nullptr) > (size_t)NGC_STATIC_SCRATCH_BYTES)
    return NGC_ERR_STATIC_SCRATCH;
  // Every GPU has its own copy of the array, at its own address: look it up once per device while that
  // device is current (in host code the array's name is only a stand-in for the symbol, not an address).
  int dev = -1;
  const int rc = g_static_scratch_once.run([&] {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    void* addr = nullptr;
    if (e == cudaSuccess) e = cudaGetSymbolAddress(&addr, g_static_scratch);
    if (e == cudaSuccess) g_static_scratch_addr[cur] = addr;
    return e;
  }, &dev);
  if (rc != NGC_OK) return rc;
  // The scratch used is the current device's: a stream of another device would make the kernels write
  // through an address that means something else there.
  int stream_dev = -1;
  NGC_CUDA_TRY(cudaStreamGetDevice((cudaStream_t)stream, &stream_dev));
  if (stream_dev != dev) return NGC_ERR_INVALID_ARG;
  return ngc_decode_attn_ragged(c, q, new_k, new_v, layer_begin, layer_end, scale, out, out_dtype,
                                g_static_scratch_addr[dev], (size_t)NGC_STATIC_SCRATCH_BYTES, dev_status, stream);
}
