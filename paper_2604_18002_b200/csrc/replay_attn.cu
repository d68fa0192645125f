// ngc_replay_attn, warp-level MMA path (kept as the comparison arm of the tcgen05 kernel in
// replay_attn_umma.cu, which is what ngc_replay_attn runs): attention of EVERY token of a rollout
// under its replay mask (paper Section 4.5 and Appendix A.3): one pass over the full, uncompacted sequence in which the query at position t
// sees what it saw at generation time -- the entries the last eviction round before t left alive
// (kept_r, a list of original positions from ngc_replay_visibility) plus, causally, the tokens
// generated since that round.  The paper feeds dense B x T x T masks to a stock attention; here the
// kept list is GATHERED, so the work is proportional to what is visible, not to T^2.
//
// bf16, d = 128.  One CTA per (layer, sequence, query head, 64 query tokens), four warps of 16
// query rows; keys and values arrive in 64-row tiles through a double-buffered cp.async pipeline
// (rows of the kept list gathered by position, rows of the current block contiguous), stored with
// the 128-byte XOR swizzle so that ldmatrix is conflict free.  S = Q K^T and O += P V run on the
// tensor cores (mma.sync m16n8k16, Q fragments in registers, P re-used from the accumulators),
// single-pass online softmax in fp32, log2 domain.  A 64-token query tile may straddle eviction
// rounds: every query row carries its own block index and lower bound, applied as a mask.
#include <cuda_bf16.h>

#include "ngc_common.cuh"
#include "ptx.cuh"
#include "replay_attn.cuh"

namespace ngc {
namespace {

constexpr int kQTile = 64;                    // query tokens per CTA
constexpr int kKTile = 64;                    // keys per pipeline stage
constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kBoxBytes = kKTile * 128;       // 64 rows x 64 channels of bf16
constexpr int kTileBytes = 2 * kBoxBytes;     // K (or V) tile
constexpr int kStageBytes = 2 * kTileBytes;   // K + V
constexpr int kMaxSeg = 66;                   // rounds one query tile can straddle (+ the contiguous part)

// swizzled byte offset of 16-byte piece c (0..15) of row r inside a K or V tile
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return (uint32_t)((c >> 3) * kBoxBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

__global__ void __launch_bounds__(kThreads, 3) replay_attn_kernel(ReplayAttnParams p) {
  extern __shared__ uint8_t smem_dyn[];
  // key sources of this query tile: the kept lists of the rounds it straddles, then the contiguous run
  __shared__ int s_seg_rho[kMaxSeg], s_seg_n[kMaxSeg], s_seg_first[kMaxSeg + 1];
  __shared__ int s_nseg, s_clo, s_uniform;

  uint8_t* stage = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;

  int item = blockIdx.x;
  const int m = item % p.q_tiles; item /= p.q_tiles;
  const int hq = item % p.Hq; item /= p.Hq;
  const int b = item % p.B;
  const int l = item / p.B;
  const int T_b = min(p.lens[b], p.t_max);
  const int q0 = m * kQTile;
  if (q0 >= T_b) return;
  const int h = hq / p.g;
  const int gi = list_of(p.lists, l, h, p.Hkv);
  const int q_last = min(q0 + kQTile - 1, T_b - 1);

  if (tid == 0) {
    int r_lo = 0, r_hi = 0;                       // rounds fired before the first / last query of the tile
    for (int r = 0; r < p.n_rounds; ++r) {
      const int tb = p.total_before[r * p.B + b];
      r_lo += tb <= q0;
      r_hi += tb <= q_last;
    }
    int nseg = 0, first = 0;
    for (int rho = max(r_lo, 1); rho <= r_hi && nseg < kMaxSeg - 1; ++rho) {
      int n = p.alive_count[((int64_t)(rho - 1) * p.B + b) * p.G + gi];
      if (n < 0 || n > p.kt_max) { set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT); n = 0; }
      if (n > 0) {
        s_seg_rho[nseg] = rho; s_seg_n[nseg] = n; s_seg_first[nseg] = first;
        first += (n + kKTile - 1) / kKTile;
        ++nseg;
      }
    }
    const int c_lo = r_lo >= 1 ? p.total_before[(r_lo - 1) * p.B + b] : 0;
    s_clo = c_lo;
    s_seg_rho[nseg] = -1; s_seg_n[nseg] = q_last - c_lo + 1; s_seg_first[nseg] = first;
    first += (q_last - c_lo + kKTile) / kKTile;
    ++nseg;
    s_seg_first[nseg] = first;
    s_nseg = nseg;
    s_uniform = r_lo == r_hi;                     // every query of the tile lies in the same block
  }
  __syncthreads();
  const int nseg = s_nseg, c_lo = s_clo, n_tiles = s_seg_first[nseg];
  const bool uniform = s_uniform != 0;

  // this thread's two query rows: position, round index, first position of its own block
  const int t_row[2] = {q0 + 16 * warp + gid, q0 + 16 * warp + gid + 8};
  int blk[2] = {0, 0}, lo_row[2] = {0, 0};
  for (int r = 0; r < p.n_rounds; ++r) {
    const int tb = p.total_before[r * p.B + b];
#pragma unroll
    for (int e = 0; e < 2; ++e)
      if (tb <= t_row[e]) { blk[e] += 1; lo_row[e] = tb; }
  }
  // Q fragments (A operand): rows gid, gid + 8 of this warp's 16 query tokens
  uint32_t qa[8][4];
  {
    const uint32_t* qbase = (const uint32_t*)(p.q + (((int64_t)l * p.B + b) * p.Hq + hq) * (int64_t)p.t_max * 128);
    const bool v0 = t_row[0] < T_b, v1 = t_row[1] < T_b;
    const uint32_t* r0 = qbase + (int64_t)t_row[0] * 64;
    const uint32_t* r1 = qbase + (int64_t)t_row[1] * 64;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = v0 ? r0[8 * ks + tig] : 0u;
      qa[ks][1] = v1 ? r1[8 * ks + tig] : 0u;
      qa[ks][2] = v0 ? r0[8 * ks + tig + 4] : 0u;
      qa[ks][3] = v1 ? r1[8 * ks + tig + 4] : 0u;
    }
  }
  const __nv_bfloat16* k_strip = p.k + ((int64_t)(l * p.Hkv + h) * p.rows_R + p.seq_off[b]) * 128;
  const __nv_bfloat16* v_strip = p.v + ((int64_t)(l * p.Hkv + h) * p.rows_R + p.seq_off[b]) * 128;
  const uint32_t stage_u32 = ptx::smem_u32(stage);

  // ---- loader: tile i of the key sequence into buffer i & 1 (every thread moves 8 pieces of K and of V)
  auto load_tile = [&](int i) {
    int sgi = 0;
    while (sgi + 1 < nseg && i >= s_seg_first[sgi + 1]) ++sgi;
    const int rho = s_seg_rho[sgi], n = s_seg_n[sgi], kt = i - s_seg_first[sgi];
    const int32_t* list = rho >= 1 ? p.alive_pos + (((int64_t)(rho - 1) * p.B + b) * p.G + gi) * p.kt_max : nullptr;
    const uint32_t buf = stage_u32 + (uint32_t)(i & 1) * kStageBytes;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int slot = u * kThreads + tid;
      const int row = slot >> 4, c = slot & 15;
      const int kidx = kt * kKTile + row;
      int pos = -1;
      if (kidx < n) pos = list ? list[kidx] : c_lo + kidx;
      const uint32_t off = tile_off(row, c);
      if (pos >= 0 && pos < T_b) {
        ptx::cp_async_cg_16(buf + off, k_strip + (int64_t)pos * 128 + 8 * c);
        ptx::cp_async_cg_16(buf + kTileBytes + off, v_strip + (int64_t)pos * 128 + 8 * c);
      } else {        // past the end of the source: zeros (a stale NaN times P = 0 would poison the sum)
        if (kidx < n && c == 0) set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT);
        *reinterpret_cast<uint4*>(stage + (i & 1) * kStageBytes + off) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(stage + (i & 1) * kStageBytes + kTileBytes + off) = make_uint4(0, 0, 0, 0);
      }
    }
  };

  float o_acc[16][4];
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < 16; ++i) { o_acc[i][0] = 0.f; o_acc[i][1] = 0.f; o_acc[i][2] = 0.f; o_acc[i][3] = 0.f; }
  const uint32_t x7 = (uint32_t)(lane & 7);
  const uint32_t kb_row = (uint32_t)((lane & 7) + 8 * (lane >> 4));          // K rows as B operand of S
  const uint32_t vb_row = (uint32_t)((lane & 7) + 8 * ((lane >> 3) & 1));    // V rows as B operand of O

  load_tile(0);
  ptx::cp_async_commit();
  for (int i = 0; i < n_tiles; ++i) {
    if (i + 1 < n_tiles) load_tile(i + 1);
    ptx::cp_async_commit();
    ptx::cp_async_wait_group<1>();
    __syncthreads();

    int sgi = 0;
    while (sgi + 1 < nseg && i >= s_seg_first[sgi + 1]) ++sgi;
    const int rho = s_seg_rho[sgi], kt = i - s_seg_first[sgi];
    const int n_here = min(kKTile, s_seg_n[sgi] - kt * kKTile);
    const uint32_t k_st = stage_u32 + (uint32_t)(i & 1) * kStageBytes;
    const uint32_t v_st = k_st + kTileBytes;

    // ---- S = Q K^T: 16 query rows x 64 keys ----
    float sc[8][4];
#pragma unroll
    for (int n8 = 0; n8 < 8; ++n8) { sc[n8][0] = 0.f; sc[n8][1] = 0.f; sc[n8][2] = 0.f; sc[n8][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t chunk = (uint32_t)(2 * (ks & 3) + ((lane >> 3) & 1));
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t r0, r1, r2, r3;
        ptx::ldmatrix_x4(k_st + (ks >> 2) * kBoxBytes + (16 * np + kb_row) * 128 + ((chunk ^ x7) << 4), r0, r1, r2, r3);
        ptx::mma_bf16_16816(sc[2 * np], qa[ks], r0, r1);
        ptx::mma_bf16_16816(sc[2 * np + 1], qa[ks], r2, r3);
      }
    }
    // ---- visibility and online softmax (log2 domain) ----
    // a tile needs no mask when every query of the CTA lies in one block and the tile is a full
    // tile of that block's kept list, or lies entirely before the first query
    const bool need_mask = !uniform || (rho >= 1 ? n_here < kKTile : c_lo + kt * kKTile + kKTile - 1 > q0);
    float mx[2] = {-INFINITY, -INFINITY};
    if (need_mask) {
#pragma unroll
      for (int n8 = 0; n8 < 8; ++n8)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int jj = 8 * n8 + 2 * tig + (e & 1), r = e >> 1;
          bool vis;
          if (rho >= 1) {
            vis = jj < n_here && blk[r] == rho;                       // a kept entry of the round before this row's block
          } else {
            const int j = c_lo + kt * kKTile + jj;                    // a token of the row's own block, causal
            vis = j >= lo_row[r] && j <= t_row[r];
          }
          const float z = vis ? sc[n8][e] * p.scale_log2 : -INFINITY;
          sc[n8][e] = z;
          mx[r] = fmaxf(mx[r], z);
        }
    } else {
#pragma unroll
      for (int n8 = 0; n8 < 8; ++n8)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          sc[n8][e] *= p.scale_log2;
          mx[e >> 1] = fmaxf(mx[e >> 1], sc[n8][e]);
        }
    }
    float alpha[2], m_use[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);
      m_use[r] = m_new == -INFINITY ? 0.f : m_new;                  // nothing visible yet: exponents of -inf give 0
      alpha[r] = ptx::ex2_approx(m_run[r] - m_use[r]);
      m_run[r] = m_new;
      l_run[r] *= alpha[r];
    }
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      o_acc[n][0] *= alpha[0]; o_acc[n][1] *= alpha[0];
      o_acc[n][2] *= alpha[1]; o_acc[n][3] *= alpha[1];
    }
    uint32_t pa[4][4];
#pragma unroll
    for (int n8 = 0; n8 < 8; ++n8) {
      float pr[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        pr[e] = ptx::ex2_approx(sc[n8][e] - m_use[e >> 1]);
        l_run[e >> 1] += pr[e];
      }
      pa[n8 >> 1][2 * (n8 & 1)] = ptx::pack_bf16x2(pr[0], pr[1]);
      pa[n8 >> 1][2 * (n8 & 1) + 1] = ptx::pack_bf16x2(pr[2], pr[3]);
    }
    // ---- O += P V: 16 rows x 128 channels over the 64 keys ----
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int np = 0; np < 8; ++np) {
        const uint32_t chunk = (uint32_t)(2 * (np & 3) + (lane >> 4));
        uint32_t r0, r1, r2, r3;
        ptx::ldmatrix_x4_trans(v_st + (np >> 2) * kBoxBytes + (16 * kk + vb_row) * 128 + ((chunk ^ x7) << 4), r0, r1, r2, r3);
        ptx::mma_bf16_16816(o_acc[2 * np], pa[kk], r0, r1);
        ptx::mma_bf16_16816(o_acc[2 * np + 1], pa[kk], r2, r3);
      }
    }
    __syncthreads();          // the buffer is refilled by the load issued in the next iteration
  }
  // ---- normalise and write the rows that exist ----
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (t_row[r] >= T_b) continue;
    const float inv = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
    const int64_t base = ((((int64_t)l * p.B + b) * p.Hq + hq) * (int64_t)p.t_max + t_row[r]) * 128 + 2 * tig;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      const float x = o_acc[n][2 * r] * inv, y = o_acc[n][2 * r + 1] * inv;
      if (p.out_bf16) *reinterpret_cast<uint32_t*>((__nv_bfloat16*)p.out + base + 8 * n) = ptx::pack_bf16x2(x, y);
      else *reinterpret_cast<float2*>((float*)p.out + base + 8 * n) = make_float2(x, y);
    }
  }
}

}  // namespace
}  // namespace ngc

namespace ngc {
namespace {

int replay_attn_impl(const ngc_cache* c, const void* q, int t_max,
                     const int32_t* alive_pos, const int32_t* alive_count, const int32_t* total_before,
                     int n_rounds, int kt_max, int lists, float scale, void* out, int out_dtype, int variant,
                     int32_t* dev_status, cudaStream_t stream) {
  if (!valid_cache(c) || !q || !out || t_max <= 0 || n_rounds < 0 || lists < 0 || lists > 2 || variant < 0 || variant > 2 ||
      (n_rounds > 0 && (!alive_pos || !alive_count || !total_before || kt_max <= 0)))
    return NGC_ERR_INVALID_ARG;
  if (out_dtype != NGC_F32 && out_dtype != NGC_BF16) return NGC_ERR_INVALID_ARG;
  if (c->dtype != NGC_BF16 || c->d != 128) return NGC_ERR_UNSUPPORTED;
  if (c->lens_lists != 0) return NGC_ERR_INVALID_ARG;      // the full sequences have one length each
  if ((((uintptr_t)c->k | (uintptr_t)c->v | (uintptr_t)q | (uintptr_t)out) & 15) != 0) return NGC_ERR_INVALID_ARG;
  if (c->rows == 0) return NGC_OK;
  ReplayAttnParams p;
  p.k = (const __nv_bfloat16*)c->k; p.v = (const __nv_bfloat16*)c->v; p.seq_off = c->seq_off; p.lens = c->lens;
  p.q = (const __nv_bfloat16*)q; p.alive_pos = alive_pos; p.alive_count = alive_count; p.total_before = total_before;
  p.out = out; p.dev_status = dev_status; p.rows_R = c->rows;
  p.L = c->L; p.B = c->B; p.Hq = c->Hq; p.Hkv = c->Hkv; p.g = c->Hq / c->Hkv; p.t_max = t_max; p.n_rounds = n_rounds;
  p.G = lists_G(lists, c->L, c->Hkv); p.kt_max = kt_max; p.lists = lists; p.out_bf16 = out_dtype == NGC_BF16;
  p.q_tiles = (t_max + kQTile - 1) / kQTile;
  p.scale_log2 = scale * 1.4426950408889634f;
  // the tcgen05 kernel takes row maxima on the raw scores, which needs a positive scale; anything else (and an
  // explicit request) runs on the warp-level kernel
  if (variant == NGC_REPLAY_ATTN_TCGEN05 && !(scale > 0.f)) return NGC_ERR_UNSUPPORTED;
  if (variant != NGC_REPLAY_ATTN_MMA_SYNC && scale > 0.f) return launch_replay_attn_umma(p, stream);
  const int64_t ctas = (int64_t)c->L * c->B * c->Hq * p.q_tiles;
  if (ctas > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  const int smem = 2 * kStageBytes + 1024;
  NGC_CUDA_TRY(cudaFuncSetAttribute(replay_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  replay_attn_kernel<<<(unsigned)ctas, kThreads, smem, stream>>>(p);
  return launch_status();
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_replay_attn(const ngc_cache* c, const void* q, int t_max,
                               const int32_t* alive_pos, const int32_t* alive_count, const int32_t* total_before,
                               int n_rounds, int kt_max, int lists, float scale, void* out, int out_dtype,
                               int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_replay_attn");
  return ngc::replay_attn_impl(c, q, t_max, alive_pos, alive_count, total_before, n_rounds, kt_max, lists, scale, out, out_dtype,
                               NGC_REPLAY_ATTN_AUTO, dev_status, (cudaStream_t)stream);
}

extern "C" int ngc_replay_attn_variant(const ngc_cache* c, const void* q, int t_max,
                                       const int32_t* alive_pos, const int32_t* alive_count, const int32_t* total_before,
                                       int n_rounds, int kt_max, int lists, float scale, void* out, int out_dtype, int variant,
                                       int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_replay_attn_variant");
  return ngc::replay_attn_impl(c, q, t_max, alive_pos, alive_count, total_before, n_rounds, kt_max, lists, scale, out, out_dtype,
                               variant, dev_status, (cudaStream_t)stream);
}
