// Gradient pass of ngc_score_evict_backward on the 5th-generation tensor cores (scores of paper
// Section 4.2, differentiated for the eviction loss of Section 4.4).
//
// With the row statistics of the first pass (maximum, sum of exponentials, c[r] = sum_t A[r][t] P[t]) the pass
// streams K once more and forms, per tile of 128 tokens (the 128 lanes of tensor memory),
//   S   [token][r]  = K Q^T                       tcgen05.mma, M = 128, N = rows padded to 16 / 32 / 48, K = 128
//   dz  [token][r]  = A (P[token] - c[r]) / sqrt(d)   one thread per token, S row read with tcgen05.ld
//   dK  [token][ch] = dz Q                        dz as the A operand FROM TENSOR MEMORY (bf16 pairs written over
//                                                 the S columns), Q as MN-major B operand
//   dQ^T[ch][r]    += K^T dz                      K tile as MN-major A operand, dz from shared memory (MN-major B);
//                                                 accumulated in tensor memory over the item's tiles
// so K is read once, dK written once and nothing else touches HBM.  The kernel is persistent, one CTA per SM
// walking the items (strip, token range) blockIdx.x, blockIdx.x + gridDim.x, ...; its warps are roles that meet
// at mbarriers only:
//   warp 0      TMA producer: K tiles (two 64-channel boxes of 128 tokens) into a 4-stage ring, running ahead
//               across item boundaries;
//   warp 1      one thread issues every MMA: S of tile t+1 before dK / dQ of tile t, so the tensor pipe works on
//               the next S while the dz of the current tile is being formed;
//   warps 2-5   dz: thread per token; at item boundaries the same warps store the finished dQ^T partial, load the
//               next item's query rows into shared memory (swizzled, zero padded) and merge its row statistics;
//   warps 6-9   dK: tensor memory -> bf16 -> swizzled shared memory -> one TMA tensor store per 64-channel box
//               (the strip's last, partly filled tile is stored row by row: rows beyond the sequence stay untouched).
// Every wait is bounded: a wait that runs out raises a CTA-wide abort flag, every role leaves its loops, copies in
// flight are waited for (bounded again), tensor memory is freed and NGC_DEV_TIMEOUT is reported.
#include <cuda.h>
#include <cuda_bf16.h>

#include "kv_map.cuh"
#include "ngc_common.cuh"
#include "ptx.cuh"
#include "score_backward.cuh"
#include "umma.cuh"

namespace ngc {
namespace {

constexpr int kTok = 128;                         // tokens per tile = tensor-memory lanes
constexpr int kStages = 4;
constexpr int kBox = kTok * 128;                  // 128 tokens x 64 channels of bf16
constexpr int kStageBytes = 2 * kBox;             // 32 KB
constexpr int kQRowsPad = 48;
constexpr int kQBox = kQRowsPad * 128;            // 48 rows x 64 channels
constexpr int kQBytes = 2 * kQBox;
constexpr int kDzBytes = kTok * 128;              // dz of a tile as B operand: [token][64 rows of bf16], 128-byte swizzle
constexpr int kSmemBytes = kStages * kStageBytes + kQBytes + 2 * kDzBytes + kStageBytes + 1024;
constexpr int kProducerWarp = 0, kMmaWarp = 1, kDzWarp0 = 2, kDkWarp0 = 6;
constexpr int kThreads = 10 * 32;
constexpr uint32_t kTmemCols = 512;               // S / dz [2] at 64 b, dK [2] at 128 + 128 b, dQ^T at 384 (64 columns)
constexpr uint32_t kTmemDk = 128, kTmemDq = 384;

struct Shared {
  uint64_t k_full[kStages], k_empty[kStages], s_full[2], dz_full[2], dzs_empty[2], dk_full[2], dk_empty[2];
  uint64_t q_ready, dq_full, drain;
  uint32_t tmem;
  int abort;
  float4 rowc[kQRowsPad];                         // per row of the item: exponent offset, c[r], last visible token, -
};

// Bounded wait that also gives up as soon as another thread of the CTA has given up.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, int* abort_flag, int32_t* dev_status) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  for (uint32_t spins = 0;; ++spins) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((spins & 63u) == 63u) {
      if (*(volatile int*)abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
        *(volatile int*)abort_flag = 1;
        set_dev_status(dev_status, NGC_DEV_TIMEOUT);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, int* abort_flag, int32_t* dev_status) {
  return __all_sync(0xffffffffu, wait_or_abort(bar, parity, abort_flag, dev_status));
}

// One item: a token range of one strip, in tiles of 128 tokens.
struct Item { int split, strip, h, b, l, T_b, tile_lo, n_tiles, gi; };
__device__ __forceinline__ Item decode_item(const BwdParams& p, int item) {
  Item it;
  it.split = item % p.n_split;
  it.strip = item / p.n_split;
  it.h = it.strip % p.Hkv;
  it.b = (it.strip / p.Hkv) % p.B;
  it.l = it.strip / (p.Hkv * p.B);
  it.T_b = p.lens[len_index(p.lens_lists, p.L, p.Hkv, it.b, it.l, it.h)];
  const int nt = (it.T_b + kTok - 1) / kTok;
  const int tps = (nt + p.n_split - 1) / p.n_split;
  it.tile_lo = min(nt, it.split * tps);
  it.n_tiles = min(nt, it.tile_lo + tps) - it.tile_lo;
  it.gi = list_of(p.lists, it.l, it.h, p.Hkv);
  return it;
}

// Named barriers of one 128-thread role.  group_all also makes the role agree on whether to go on: every thread
// gets the AND of all predicates, so that nobody waits at a later bar_sync for a warp that has given up.
__device__ __forceinline__ void bar_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
__device__ __forceinline__ bool group_all(int id, bool pred) {
  uint32_t r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %2, 0;\n\tbar.red.and.pred p, %1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(r) : "r"(id), "r"((uint32_t)pred) : "memory");
  return r != 0;
}

struct Maps { CUtensorMap k, gk; };

template <int NC>      // rows padded to the MMA's N: 16, 32 or 48
__global__ void __launch_bounds__(kThreads, 1)
score_bwd_umma_kernel(const __grid_constant__ Maps maps, BwdParams p, int n_items) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ Shared sh;

  uint8_t* base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  uint8_t* stage = base;                                 // [kStages][2 boxes of 128 tokens x 64 channels]
  uint8_t* sQ = stage + kStages * kStageBytes;           // [2 boxes][48 rows x 64 channels]
  uint8_t* sDz = sQ + kQBytes;                           // [2][128 tokens x 64 rows]
  uint8_t* sDk = sDz + 2 * kDzBytes;                     // [2 boxes][128 tokens x 64 channels] on their way out
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&sh.k_full[s], 1); ptx::mbar_init(&sh.k_empty[s], 1); }
#pragma unroll
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&sh.s_full[b], 1); ptx::mbar_init(&sh.dz_full[b], 128); ptx::mbar_init(&sh.dzs_empty[b], 1);
      ptx::mbar_init(&sh.dk_full[b], 1); ptx::mbar_init(&sh.dk_empty[b], 128);
    }
    ptx::mbar_init(&sh.q_ready, 128);
    ptx::mbar_init(&sh.dq_full, 1);
    ptx::mbar_init(&sh.drain, 1);
    ptx::fence_barrier_init();
    sh.abort = 0;
    ptx::prefetch_tensormap(&maps.k);
    ptx::prefetch_tensormap(&maps.gk);
  }
  // the dz tiles' unused rows (NC .. 63) are zero for the whole launch
  for (int x = tid; x < 2 * kDzBytes / 16; x += kThreads) reinterpret_cast<uint4*>(sDz)[x] = make_uint4(0, 0, 0, 0);
  ptx::fence_proxy_async();
  if (warp == kMmaWarp) umma::tmem_alloc(&sh.tmem, kTmemCols);
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem = sh.tmem;

  // Every role walks the same items in the same order and keeps its own running tile count: tile t (over all items)
  // uses K stage t % 4, S / dz / dK buffer t & 1.

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer: K tiles by TMA
    if (lane == 0) {
      int t = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const Item it = decode_item(p, item);
        const int plane = it.l * p.Hkv + it.h;
        const int row0 = (int)p.seq_off[it.b];
        for (int i = 0; i < it.n_tiles; ++i, ++t) {
          const int s = t % kStages;
          if (t >= kStages && !wait_or_abort(&sh.k_empty[s], ((t / kStages) - 1) & 1, &sh.abort, p.dev_status)) { ok = false; break; }
          uint8_t* sp = stage + s * kStageBytes;
          ptx::mbar_expect_tx(&sh.k_full[s], kStageBytes);
          const int y = row0 + (it.tile_lo + i) * kTok;
          ptx::tma_load_3d(sp, &maps.k, 0, y, plane, &sh.k_full[s]);
          ptx::tma_load_3d(sp + kBox, &maps.k, 64, y, plane, &sh.k_full[s]);
        }
      }
      // loads still in flight land before the CTA's shared memory goes away (only an aborted run has any)
      for (int u = max(0, t - kStages); u < t; ++u) ptx::mbar_wait_bounded(&sh.k_full[u % kStages], (u / kStages) & 1);
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma::instr_desc(kTok, NC, false);
      constexpr uint32_t idesc_dk = umma::instr_desc(kTok, 128, true);
      constexpr uint32_t idesc_dq = umma::instr_desc(128, 64, true, true);
      const uint64_t desc_hi = (uint64_t)umma::smem_desc_sw128(0, 0, 1024) & 0xffffffff00000000ull;
      const uint32_t st_addr = ptx::smem_u32(stage);
      const uint32_t q_lo = (ptx::smem_u32(sQ) >> 4) | (1u << 16);                        // K-major: leading offset unused
      const uint32_t q_mn_lo = (ptx::smem_u32(sQ) >> 4) | ((uint32_t)(kQBox >> 4) << 16);  // MN-major: next 64 channels one box on
      const uint32_t dz_addr = ptx::smem_u32(sDz);
      int t = 0, nq = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const Item it = decode_item(p, item);
        const int n = it.n_tiles;
        if (n == 0) continue;
        ok = wait_or_abort(&sh.q_ready, nq & 1, &sh.abort, p.dev_status);      // Q rows in place, dQ^T of the previous item read
        if (!ok) break;
        umma::fence_after_sync();
        auto issue_s = [&](int tt) {                                   // S = K Q^T of tile tt into S buffer tt & 1
          const uint32_t k_lo = ((st_addr + (tt % kStages) * kStageBytes) >> 4) | (1u << 16);
          const uint32_t d = tmem + (uint32_t)(64 * (tt & 1));
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint64_t a = desc_hi | (uint64_t)(k_lo + (uint32_t)(((ks >> 2) * kBox + (ks & 3) * 32) >> 4));
            const uint64_t b = desc_hi | (uint64_t)(q_lo + (uint32_t)(((ks >> 2) * kQBox + (ks & 3) * 32) >> 4));
            umma::mma_bf16(d, a, b, idesc_s, ks > 0);
          }
          umma::commit(&sh.s_full[tt & 1]);
        };
        ok = wait_or_abort(&sh.k_full[t % kStages], (t / kStages) & 1, &sh.abort, p.dev_status);
        if (!ok) break;
        issue_s(t);
        for (int i = 0; i < n; ++i) {
          const int tt = t + i, buf = tt & 1;
          if (i + 1 < n) {
            ok = wait_or_abort(&sh.k_full[(tt + 1) % kStages], ((tt + 1) / kStages) & 1, &sh.abort, p.dev_status);
            if (!ok) break;
            issue_s(tt + 1);      // its buffer held S and dz of tile tt - 1, whose dK product was issued before this one
          }
          ok = wait_or_abort(&sh.dz_full[buf], (tt >> 1) & 1, &sh.abort, p.dev_status);
          if (ok && tt >= 2) ok = wait_or_abort(&sh.dk_empty[buf], ((tt >> 1) - 1) & 1, &sh.abort, p.dev_status);
          if (!ok) break;
          umma::fence_after_sync();
          // dK = dz Q: 16 rows per step = 8 packed columns of dz, two 8-row groups of Q
#pragma unroll
          for (int kk = 0; kk < NC / 16; ++kk)
            umma::mma_bf16_a_tmem(tmem + kTmemDk + 128u * buf, tmem + 64u * buf + 8u * kk,
                                  desc_hi | (uint64_t)(q_mn_lo + (uint32_t)((kk * 2048) >> 4)), idesc_dk, kk > 0);
          umma::commit(&sh.dk_full[buf]);
          // dQ^T += K^T dz: 16 tokens per step = two 8-row groups of the K tile and of the dz tile
          const uint32_t kt_lo = ((st_addr + (tt % kStages) * kStageBytes) >> 4) | ((uint32_t)(kBox >> 4) << 16);
          const uint32_t dz_lo = ((dz_addr + buf * kDzBytes) >> 4) | (1u << 16);
#pragma unroll
          for (int kt = 0; kt < 8; ++kt)
            umma::mma_bf16(tmem + kTmemDq, desc_hi | (uint64_t)(kt_lo + (uint32_t)((kt * 2048) >> 4)),
                           desc_hi | (uint64_t)(dz_lo + (uint32_t)((kt * 2048) >> 4)), idesc_dq, (i > 0 || kt > 0) ? 1u : 0u);
          umma::commit(&sh.k_empty[tt % kStages]);
          umma::commit(&sh.dzs_empty[buf]);
          if (i + 1 == n) umma::commit(&sh.dq_full);
        }
        t += n;
        ++nq;
      }
      umma::commit(&sh.drain);          // everything issued has completed before tensor memory is released
      wait_or_abort(&sh.drain, 0, &sh.abort, p.dev_status);
    }
    __syncwarp();
  } else if (warp < kDkWarp0) {
    // ------------------------------------------------------------------ dz: one thread per token
    const int row = 32 * (warp & 3) + lane;                            // token of the tile = tensor-memory lane = channel of dQ^T
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const int gtid = tid - kDzWarp0 * 32;                              // 0 .. 127
    int t = 0, nq = 0;
    bool ok = true;
    float* prev_part = nullptr;                                        // where the dQ^T in tensor memory belongs
    auto flush_dq = [&]() {                                            // the finished item's dQ partial: rows x 128 channels, fp32
      if (!warp_wait(&sh.dq_full, (nq - 1) & 1, &sh.abort, p.dev_status)) return false;
      umma::fence_after_sync();
      uint32_t v[NC];
#pragma unroll
      for (int c = 0; c < NC; c += 16) umma::tmem_ld16(tmem + lane_base + kTmemDq + c, v + c);
      umma::tmem_ld_wait();
#pragma unroll
      for (int r = 0; r < NC; ++r)
        if (r < p.n_rows) prev_part[r * 128 + row] = __uint_as_float(v[r]);
      umma::fence_before_sync();
      return true;
    };
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
      const Item it = decode_item(p, item);
      // with one token range per strip the partial is the gradient itself (the strip's rows are contiguous in grad_q)
      float* part = p.n_split == 1 ? p.grad_q + ((((int64_t)it.l * p.B + it.b) * p.Hq + it.h * p.g) * p.w) * 128
                                   : p.dq_part + ((int64_t)it.strip * p.n_split + it.split) * kBwdMaxRows * 128;
      if (it.n_tiles == 0) {                                           // an empty range still owns a partial
        for (int r = 0; r < p.n_rows; ++r) part[r * 128 + row] = 0.f;
        continue;
      }
      const int T_b = it.T_b;
      // ---- item set-up: query rows and row statistics are fetched before the previous item's dQ^T is waited for
      uint4 qv[6];
#pragma unroll
      for (int u = 0; u < 6; ++u) {
        const int x = gtid + 128 * u, r = x >> 4, piece = x & 15;      // 48 rows x 16 pieces of 16 bytes
        qv[u] = make_uint4(0, 0, 0, 0);
        if (r < p.n_rows)
          qv[u] = ((const uint4*)((const __nv_bfloat16*)p.q_recent +
                                  ((((int64_t)it.l * p.B + it.b) * p.Hq + it.h * p.g) * p.w + r) * 128))[piece];
      }
      float4 rc = make_float4(-INFINITY, 0.f, __int_as_float(-1), 0.f);
      if (gtid < p.n_rows) {
        const float4* st = p.stats + (int64_t)it.strip * p.n_split * kBwdMaxRows;
        float m = -INFINITY, sum = 0.f, num = 0.f;
        for (int c = 0; c < p.n_split; ++c) {
          const float4 v = st[c * kBwdMaxRows + gtid];
          merge3(m, sum, num, v.x, v.y, v.z);
        }
        if (sum > 0.f) rc = make_float4(-m + log2f(p.inv_sqrt_d / sum), num / sum, __int_as_float(column_limit(p, gtid, T_b)), 0.f);
      }
      if (nq > 0) ok = flush_dq();
      ok = group_all(1, ok);
      if (!ok) break;
      prev_part = part;
#pragma unroll
      for (int u = 0; u < 6; ++u) {
        const int x = gtid + 128 * u, r = x >> 4, piece = x & 15;
        *reinterpret_cast<uint4*>(sQ + (piece >> 3) * kQBox + r * 128 + (((piece & 7) ^ (r & 7)) << 4)) = qv[u];
      }
      if (gtid < kQRowsPad) sh.rowc[gtid] = rc;
      ptx::fence_proxy_async();                                        // the MMAs read Q through the async proxy
      ptx::mbar_arrive(&sh.q_ready);
      bar_sync(1);                                                     // rowc is visible to the four warps
      ++nq;
      const float inv_rows = inv_list_rows(p, T_b);
      // upstream weights: loaded one tile ahead, turned into P at the end of the tile before
      float P_next = token_weight_finish(p, token_weight_issue(p, it.b, it.gi, it.tile_lo * kTok + row, T_b, inv_rows));
      for (int i = 0; i < it.n_tiles; ++i) {
        const int tt = t + i, buf = tt & 1;
        const int t_tile = (it.tile_lo + i) * kTok;
        const int t_tok = t_tile + row;
        const float P = P_next;
        const TokenWeightRaw raw_next = token_weight_issue(p, it.b, it.gi, i + 1 < it.n_tiles ? t_tok + kTok : T_b, T_b, inv_rows);
        if (!warp_wait(&sh.s_full[buf], (tt >> 1) & 1, &sh.abort, p.dev_status)) { ok = false; break; }
        umma::fence_after_sync();
        uint32_t sv[NC];
        const uint32_t s_addr = tmem + lane_base + 64u * buf;
#pragma unroll
        for (int c = 0; c < NC; c += 16) umma::tmem_ld16(s_addr + c, sv + c);
        umma::tmem_ld_wait();
        const bool masked = t_tile + kTok > T_b - p.w;                 // some row cannot see some token of this tile
        uint32_t pk[NC / 2];
#pragma unroll
        for (int r = 0; r < NC; r += 2) {
          const float4 c0 = sh.rowc[r], c1 = sh.rowc[r + 1];
          float d0 = ptx::ex2_approx(fmaf(__uint_as_float(sv[r]), p.scale_log2, c0.x)) * (P - c0.y);
          float d1 = ptx::ex2_approx(fmaf(__uint_as_float(sv[r + 1]), p.scale_log2, c1.x)) * (P - c1.y);
          if (masked) {
            d0 = t_tok <= __float_as_int(c0.z) ? d0 : 0.f;
            d1 = t_tok <= __float_as_int(c1.z) ? d1 : 0.f;
          }
          pk[r >> 1] = ptx::pack_bf16x2(d0, d1);
        }
        // the shared-memory copy below is free once the dQ^T product of two tiles ago has read it
        if (tt >= 2 && !warp_wait(&sh.dzs_empty[buf], ((tt >> 1) - 1) & 1, &sh.abort, p.dev_status)) { ok = false; break; }
        // dz over the first NC / 2 columns of the S buffer it came from: the A operand of dK ...
#pragma unroll
        for (int c = 0; c < NC / 2; c += 8) umma::tmem_st8(s_addr + c, pk + c);
        // ... and into shared memory as the B operand of dQ^T
        uint8_t* dzr = sDz + buf * kDzBytes + row * 128;
#pragma unroll
        for (int j = 0; j < NC / 8; ++j)
          *reinterpret_cast<uint4*>(dzr + ((j ^ (row & 7)) << 4)) = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
        if (t_tok >= T_b) {
          // K rows beyond the sequence may hold anything and dQ^T multiplies them by dz = 0: zero them (S has read the stage)
          uint8_t* kr = stage + (tt % kStages) * kStageBytes + row * 128;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            *reinterpret_cast<uint4*>(kr + (j << 4)) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(kr + kBox + (j << 4)) = make_uint4(0, 0, 0, 0);
          }
        }
        umma::tmem_st_wait();
        umma::fence_before_sync();
        ptx::fence_proxy_async();
        ptx::mbar_arrive(&sh.dz_full[buf]);
        P_next = token_weight_finish(p, raw_next);
      }
      t += it.n_tiles;
    }
    if (ok && nq > 0) flush_dq();
  } else {
    // ------------------------------------------------------------------ dK: tensor memory -> bf16 -> TMA store
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const bool leader = tid == kDkWarp0 * 32;
    int t = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
      const Item it = decode_item(p, item);
      const int T_b = it.T_b, plane = it.l * p.Hkv + it.h;
      const int row0 = (int)p.seq_off[it.b];
      __nv_bfloat16* gk_strip = (__nv_bfloat16*)p.grad_k + ((int64_t)plane * p.rows_R + row0) * 128;
      for (int i = 0; i < it.n_tiles; ++i) {
        const int tt = t + i, buf = tt & 1;
        const int t_tile = (it.tile_lo + i) * kTok;
        const bool full = t_tile + kTok <= T_b;
        ok = group_all(2, warp_wait(&sh.dk_full[buf], (tt >> 1) & 1, &sh.abort, p.dev_status));
        if (!ok) break;
        umma::fence_after_sync();
        const uint32_t d_addr = tmem + lane_base + kTmemDk + 128u * buf;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint8_t* so = sDk + half * kBox;
          if (full) {
            if (leader) ptx::bulk_wait_read<1>();        // the store of this half of the previous tile has read the buffer
            bar_sync(2);
          }
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            uint32_t v[32];
            umma::tmem_ld32(d_addr + 64 * half + 32 * cc, v);
            umma::tmem_ld_wait();
            if (half == 1 && cc == 1) {                   // the tile's accumulators are in registers: the buffer is free
              umma::fence_before_sync();
              ptx::mbar_arrive(&sh.dk_empty[buf]);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 w4 = make_uint4(ptx::pack_bf16x2(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1])),
                                          ptx::pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                                          ptx::pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                                          ptx::pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
              if (full)
                *reinterpret_cast<uint4*>(so + row * 128 + (((4 * cc + q) ^ (row & 7)) << 4)) = w4;
              else if (t_tile + row < T_b && NGC_IN_BOUNDS(p.dev_status, row0 + t_tile + row < p.rows_R))
                *reinterpret_cast<uint4*>(gk_strip + (int64_t)(t_tile + row) * 128 + 64 * half + 32 * cc + 8 * q) = w4;
            }
          }
          if (full) {
            ptx::fence_proxy_async();                     // written through the generic proxy, read by the TMA store
            bar_sync(2);
            if (leader && NGC_IN_BOUNDS(p.dev_status, row0 + t_tile + kTok <= p.rows_R && plane < p.L * p.Hkv)) {
              ptx::tma_store_3d(&maps.gk, 64 * half, row0 + t_tile, plane, so);
              ptx::bulk_commit();
            }
          }
        }
      }
      t += it.n_tiles;
    }
    if (leader) ptx::bulk_wait<0>();                      // the last stores have left shared memory and reached global memory
  }
  // ---- teardown: every role has left its loops; nothing of this CTA is in flight any more
  umma::fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    umma::fence_after_sync();
    umma::tmem_dealloc(tmem, kTmemCols);
  }
}

// ---------------------------------------------------------------- first pass: row statistics
//
// The transposed product S^T = Q K^T puts the rows on the lanes of tensor memory and the 128 tokens of a tile on its
// columns, so that a thread keeps the running (maximum, sum of exponentials, sum of exponentials times P) of ONE row in
// registers and walks along its tokens without any exchange between threads.  The query rows are stacked 128 / RQ
// times in the A operand (RQ = 32 or 64 rows, zero padded): copy c of a row sits on lane RQ c + r and its thread takes
// tokens (128 / copies) c ... of every tile, so all four warps share the exponentials of a tile.  The copies of a row
// are merged when the item ends.
struct StatsShared {
  uint64_t k_full[kStages], k_empty[kStages], s_full[2], s_empty[2], q_ready, drain;
  uint32_t tmem;
  int abort;
  alignas(16) float pw[2][kTok];                  // upstream weights P of the tokens of a tile (read four at a time)
  float4 part[kTok];                              // per lane: (max, sum, sum * P) at the end of an item
};
constexpr int kStatsSmemBytes = kStages * kStageBytes + kStageBytes + 1024;      // K ring + the stacked Q tile
constexpr int kStatsThreads = 6 * 32;             // producer, MMA, four statistics warps
constexpr uint32_t kStatsTmemCols = 256;          // S^T [2] at 128 b

template <int RQ>
__global__ void __launch_bounds__(kStatsThreads, 1)
score_bwd_stats_umma_kernel(const __grid_constant__ CUtensorMap map_k, BwdParams p, int n_items) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ StatsShared sh;
  constexpr int kCopies = kTok / RQ, kTpt = kTok / kCopies;      // tokens of a tile per thread

  uint8_t* base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  uint8_t* stage = base;                                 // [kStages][2 boxes of 128 tokens x 64 channels]
  uint8_t* sQ = stage + kStages * kStageBytes;           // [2 boxes][128 stacked rows x 64 channels]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&sh.k_full[s], 1); ptx::mbar_init(&sh.k_empty[s], 1); }
#pragma unroll
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&sh.s_full[b], 1); ptx::mbar_init(&sh.s_empty[b], 128); }
    ptx::mbar_init(&sh.q_ready, 128);
    ptx::mbar_init(&sh.drain, 1);
    ptx::fence_barrier_init();
    sh.abort = 0;
    ptx::prefetch_tensormap(&map_k);
  }
  if (warp == kMmaWarp) umma::tmem_alloc(&sh.tmem, kStatsTmemCols);
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem = sh.tmem;

  if (warp == kProducerWarp) {
    if (lane == 0) {
      int t = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const Item it = decode_item(p, item);
        const int plane = it.l * p.Hkv + it.h;
        const int row0 = (int)p.seq_off[it.b];
        for (int i = 0; i < it.n_tiles; ++i, ++t) {
          const int s = t % kStages;
          if (t >= kStages && !wait_or_abort(&sh.k_empty[s], ((t / kStages) - 1) & 1, &sh.abort, p.dev_status)) { ok = false; break; }
          uint8_t* sp = stage + s * kStageBytes;
          ptx::mbar_expect_tx(&sh.k_full[s], kStageBytes);
          const int y = row0 + (it.tile_lo + i) * kTok;
          ptx::tma_load_3d(sp, &map_k, 0, y, plane, &sh.k_full[s]);
          ptx::tma_load_3d(sp + kBox, &map_k, 64, y, plane, &sh.k_full[s]);
        }
      }
      for (int u = max(0, t - kStages); u < t; ++u) ptx::mbar_wait_bounded(&sh.k_full[u % kStages], (u / kStages) & 1);
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma::instr_desc(kTok, kTok, false);
      const uint64_t desc_hi = (uint64_t)umma::smem_desc_sw128(0, 0, 1024) & 0xffffffff00000000ull;
      const uint32_t st_addr = ptx::smem_u32(stage);
      const uint32_t q_lo = (ptx::smem_u32(sQ) >> 4) | (1u << 16);
      int t = 0, nq = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const Item it = decode_item(p, item);
        if (it.n_tiles == 0) continue;
        ok = wait_or_abort(&sh.q_ready, nq & 1, &sh.abort, p.dev_status);
        if (!ok) break;
        umma::fence_after_sync();
        for (int i = 0; i < it.n_tiles; ++i, ++t) {
          const int buf = t & 1, s = t % kStages;
          ok = wait_or_abort(&sh.k_full[s], (t / kStages) & 1, &sh.abort, p.dev_status);
          if (ok && t >= 2) ok = wait_or_abort(&sh.s_empty[buf], ((t >> 1) - 1) & 1, &sh.abort, p.dev_status);
          if (!ok) break;
          umma::fence_after_sync();
          const uint32_t k_lo = ((st_addr + s * kStageBytes) >> 4) | (1u << 16);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (uint32_t)(((ks >> 2) * kBox + (ks & 3) * 32) >> 4);
            umma::mma_bf16(tmem + 128u * buf, desc_hi | (uint64_t)(q_lo + off), desc_hi | (uint64_t)(k_lo + off), idesc, ks > 0);
          }
          umma::commit(&sh.s_full[buf]);
          umma::commit(&sh.k_empty[s]);
        }
        ++nq;
      }
      umma::commit(&sh.drain);
      wait_or_abort(&sh.drain, 0, &sh.abort, p.dev_status);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ statistics: one thread per (row, copy)
    const int m = 32 * (warp & 3) + lane;                              // lane of tensor memory
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const int r = m % RQ, tok_lo = (m / RQ) * kTpt;
    int t = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
      const Item it = decode_item(p, item);
      float4* out = p.stats + ((int64_t)it.strip * p.n_split + it.split) * kBwdMaxRows;
      if (it.n_tiles == 0) {
        if (m < kBwdMaxRows) out[m] = make_float4(-INFINITY, 0.f, 0.f, 0.f);
        continue;
      }
      const int T_b = it.T_b;
      const float inv_rows = inv_list_rows(p, T_b);
      // the stacked query tile: stacked row x = copy * RQ + r, 16 pieces of 16 bytes each (every S^T product of the
      // previous item has completed: its last tile has been read below)
      const __nv_bfloat16* q_rows = (const __nv_bfloat16*)p.q_recent + ((((int64_t)it.l * p.B + it.b) * p.Hq + it.h * p.g) * p.w) * 128;
      uint4 qv[RQ / 8];                                                 // RQ rows x 16 pieces over 128 threads, all loads in flight
#pragma unroll
      for (int u = 0; u < RQ / 8; ++u) {
        const int rr = (m + 128 * u) >> 4, piece = m & 15;
        qv[u] = make_uint4(0, 0, 0, 0);
        if (rr < p.n_rows) qv[u] = ((const uint4*)(q_rows + (int64_t)rr * 128))[piece];
      }
#pragma unroll
      for (int u = 0; u < RQ / 8; ++u) {
        const int rr = (m + 128 * u) >> 4, piece = m & 15;
#pragma unroll
        for (int c = 0; c < kCopies; ++c) {
          const int x = c * RQ + rr;
          *reinterpret_cast<uint4*>(sQ + (piece >> 3) * kBox + x * 128 + (((piece & 7) ^ (x & 7)) << 4)) = qv[u];
        }
      }
      sh.pw[t & 1][m] = token_weight_finish(p, token_weight_issue(p, it.b, it.gi, it.tile_lo * kTok + m, T_b, inv_rows));
      ptx::fence_proxy_async();
      ptx::mbar_arrive(&sh.q_ready);
      const int lim = column_limit(p, r, T_b);
      float m_run = -INFINITY, s_run = 0.f, n_run = 0.f;              // maximum in raw score units
      for (int i = 0; i < it.n_tiles; ++i, ++t) {
        const int buf = t & 1;
        const int t_tile = (it.tile_lo + i) * kTok;
        // the next tile's upstream weights: loads now, arithmetic and hand-over at the end of this tile
        const TokenWeightRaw raw_next = token_weight_issue(p, it.b, it.gi, i + 1 < it.n_tiles ? t_tile + kTok + m : T_b, T_b, inv_rows);
        ok = group_all(1, warp_wait(&sh.s_full[buf], (t >> 1) & 1, &sh.abort, p.dev_status));   // also: pw[buf] is complete
        if (!ok) break;
        umma::fence_after_sync();
        const bool masked = t_tile + kTok > T_b - p.w;
#pragma unroll
        for (int c0 = 0; c0 < kTpt; c0 += 32) {
          uint32_t v[32];
          umma::tmem_ld32(tmem + lane_base + 128u * buf + tok_lo + c0, v);
          umma::tmem_ld_wait();
          if (c0 + 32 == kTpt) {                          // the thread's share of the buffer is in registers
            umma::fence_before_sync();
            ptx::mbar_arrive(&sh.s_empty[buf]);
          }
          float z[32];
          float mx = m_run;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            z[j] = __uint_as_float(v[j]);
            if (masked && t_tile + tok_lo + c0 + j > lim) z[j] = -INFINITY;
            mx = fmaxf(mx, z[j]);
          }
          if (mx == -INFINITY) continue;                  // nothing visible so far
          const float neg = -mx * p.scale_log2;
          const float e_old = ptx::ex2_approx(fmaf(m_run, p.scale_log2, neg));
          float s_acc = 0.f, n_acc = 0.f;
          const float4* pw4 = reinterpret_cast<const float4*>(&sh.pw[buf][tok_lo + c0]);
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 P4 = pw4[j >> 2];
            const float e0 = ptx::ex2_approx(fmaf(z[j], p.scale_log2, neg)), e1 = ptx::ex2_approx(fmaf(z[j + 1], p.scale_log2, neg));
            const float e2 = ptx::ex2_approx(fmaf(z[j + 2], p.scale_log2, neg)), e3 = ptx::ex2_approx(fmaf(z[j + 3], p.scale_log2, neg));
            s_acc += (e0 + e1) + (e2 + e3);
            n_acc = fmaf(e0, P4.x, fmaf(e1, P4.y, fmaf(e2, P4.z, fmaf(e3, P4.w, n_acc))));
          }
          s_run = fmaf(s_run, e_old, s_acc);
          n_run = fmaf(n_run, e_old, n_acc);
          m_run = mx;
        }
        sh.pw[buf ^ 1][m] = token_weight_finish(p, raw_next);        // every thread is past the tile that used this buffer
      }
      if (!ok) break;
      // merge the copies of a row
      sh.part[m] = make_float4(m_run * p.scale_log2, s_run, n_run, 0.f);
      bar_sync(1);
      if (m < kBwdMaxRows) {
        float mm = -INFINITY, sum = 0.f, num = 0.f;
        if (m < p.n_rows) {
#pragma unroll
          for (int c = 0; c < kCopies; ++c) merge3(mm, sum, num, sh.part[c * RQ + m].x, sh.part[c * RQ + m].y, sh.part[c * RQ + m].z);
        }
        out[m] = make_float4(mm, sum, num, 0.f);
      }
      bar_sync(1);                                                      // part[] is free again
    }
  }
  umma::fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    umma::fence_after_sync();
    umma::tmem_dealloc(tmem, kStatsTmemCols);
  }
}

template <int RQ>
int launch_stats_rq(const CUtensorMap& map_k, const BwdParams& p, int64_t items, cudaStream_t stream) {
  static PerDeviceOnce attr_once;      // the shared-memory opt-in is stored per device
  static int sm_count[kMaxDevices] = {0};
  int dev = -1;
  const int rc = attr_once.run([&] {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_count[cur], cudaDevAttrMultiProcessorCount, cur);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(score_bwd_stats_umma_kernel<RQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, kStatsSmemBytes);
    return e;
  }, &dev);
  if (rc != NGC_OK) return rc;
  const int grid = (int)(items < sm_count[dev] ? items : sm_count[dev]);
  score_bwd_stats_umma_kernel<RQ><<<grid, kStatsThreads, kStatsSmemBytes, stream>>>(map_k, p, (int)items);
  return launch_status();
}

template <int NC>
int launch_nc(const Maps& maps, const BwdParams& p, int64_t items, cudaStream_t stream) {
  static PerDeviceOnce attr_once;      // the shared-memory opt-in is stored per device
  static int sm_count[kMaxDevices] = {0};
  int dev = -1;
  const int rc = attr_once.run([&] {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_count[cur], cudaDevAttrMultiProcessorCount, cur);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_bwd_umma_kernel<NC>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    return e;
  }, &dev);
  if (rc != NGC_OK) return rc;
  // one CTA per SM by construction (205 KB of shared memory, all 512 columns of tensor memory)
  const int grid = (int)(items < sm_count[dev] ? items : sm_count[dev]);
  score_bwd_umma_kernel<NC><<<grid, kThreads, kSmemBytes, stream>>>(maps, p, (int)items);
  return launch_status();
}

}  // namespace

int launch_score_bwd_umma(const BwdParams& p, const void* k, void* grad_k, int64_t rows, int planes, int64_t items, cudaStream_t stream) {
  Maps maps;
  if (!make_kv_map(&maps.k, const_cast<void*>(k), rows, planes, kTok) || !make_kv_map(&maps.gk, grad_k, rows, planes, kTok))
    return NGC_ERR_UNSUPPORTED;
  const int rc = p.n_rows <= 32 ? launch_stats_rq<32>(maps.k, p, items, stream) : launch_stats_rq<64>(maps.k, p, items, stream);
  if (rc != NGC_OK) return rc;
  if (p.n_rows <= 16) return launch_nc<16>(maps, p, items, stream);
  if (p.n_rows <= 32) return launch_nc<32>(maps, p, items, stream);
  return launch_nc<48>(maps, p, items, stream);
}

}  // namespace ngc
