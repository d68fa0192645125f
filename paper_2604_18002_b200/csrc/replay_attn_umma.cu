// ngc_replay_attn on the 5th-generation tensor cores (paper Section 4.5 replay pass, Appendix A.3 masks).
//
// The replay pass is the one compute-bound contraction of this library: every token of a rollout
// attends to the kept list of the last eviction round before it plus, causally, its own block.
// A work item is 128 query tokens of TWO query heads that share a KV head; the 128 rows of a head
// are the 128 lanes of tensor memory.  The kernel is persistent: one CTA per SM walks a strided
// list of items, and its warps are specialised roles that only meet at mbarriers, so the gathers,
// the Q load and the tile bookkeeping of the next item run under the arithmetic of the current one.
//
//   planner warp (1)     per item: which kept lists and which contiguous run the 128 queries see
//                        (a small table in a two-slot ring), then the Q tiles of both heads into
//                        shared memory by tiled TMA as soon as the previous item's last S product has
//                        read them;
//   producer warps (4)   gather 64-key K/V tiles by position (kept lists, then the contiguous block)
//                        with 16-byte cp.async into a 4-stage ring, 128-byte swizzled.  Every lane hands
//                        its copies of a tile to the stage's mbarrier with cp.async.mbarrier.arrive.noinc:
//                        the arrival fires when the copies have landed, nobody waits for it, so the
//                        producers run a full ring ahead and a tile becomes visible to the MMA warp the
//                        moment it is complete.  (Publishing from the producer after a cp.async wait
//                        ties a tile's visibility to the issue of a later tile: the ring then runs in
//                        lockstep with the consumer.  TMA row gathers, tile::gather4, were measured too:
//                        about 80 cycles per four-row instruction, one 32 KB tile per 5000 cycles.)
//   MMA warps (2 x 1 thread, one per head)
//                        S_h = Q_h K^T (tcgen05.mma, M = 128, N = 64, both operands K-major in shared
//                        memory) into a double-buffered S in tensor memory, and O_h += P_h V (M = 128,
//                        N = 128, P read from TENSOR MEMORY as the A operand, V as MN-major B operand);
//                        completion is committed to mbarriers;
//   softmax warps (2x4)  one warpgroup per head, one thread per query row: S row from tensor memory
//                        (tcgen05.ld), replay mask, online softmax in the log2 domain, P row as packed
//                        bf16 back into the first 32 columns of the S buffer it came from (tcgen05.st),
//                        so P never touches shared memory and is double-buffered with S.  The running
//                        maximum used for the exponentials only moves when the true maximum has grown
//                        by more than 8 (a factor 256, exact in bf16 / fp32), so the O accumulator in
//                        tensor memory is rescaled rarely; when it is, the row's owner does it in place
//                        (tcgen05.ld / st) after the previous P V product has completed.  At the end of
//                        an item the same thread normalises its O row and writes it out.
//
// The S product of tile t+1 is issued before the P V product of tile t, so the tensor pipe works on
// one head while the other head's rows are in the softmax.  Every wait is bounded: a wait that runs
// out raises a CTA-wide abort flag, every role leaves its loops, in-flight copies and MMAs are
// drained (bounded again), tensor memory is freed and NGC_DEV_TIMEOUT is reported.
#include <cuda.h>
#include <cuda_bf16.h>

#include "kv_map.cuh"
#include "ngc_common.cuh"
#include "ptx.cuh"
#include "replay_attn.cuh"
#include "umma.cuh"

namespace ngc {
namespace {

constexpr int kQRows = 128;                   // query tokens per item = tensor-memory lanes
constexpr int kKeys = 64;                     // keys per pipeline stage
constexpr int kStages = 4;
constexpr int kMmaWarp = 8;                   // warps 0-7: softmax (two groups of four, one query head each);
                                              // warps 8, 9: one MMA-issuing thread per head
constexpr int kPlannerWarp = 10;
constexpr int kProducerWarp0 = 11;            // warps 11 .. 14
constexpr int kProducerWarps = 4;
constexpr int kProducerLanes = kProducerWarps * 32;
constexpr int kThreads = (kProducerWarp0 + kProducerWarps) * 32;
constexpr int kQHalf = kQRows * 128;          // one 64-channel half of a Q tile (128 rows x 128 B)
constexpr int kQBytes = 2 * kQHalf;           // 32 KB per head
constexpr int kKBox = kKeys * 128;            // 64 keys x 64 channels
constexpr int kKTile = 2 * kKBox;             // K (or V) tile, 16 KB
constexpr int kStageBytes = 2 * kKTile;       // K + V
constexpr int kOutStage = 4096;                // per softmax warp: 32 rows x 32 columns of the output on their way out
constexpr int kSmemBytes = 2 * kQBytes + kStages * kStageBytes + 8 * kOutStage + 1024;
constexpr uint32_t kTmemCols = 512;           // S[h][buf] at (2h + buf) * 64 (P over its first 32 columns), O[h] at 256 + 128 h
constexpr int kMaxSeg = 34;                   // rounds one query tile can straddle (+ the contiguous part)
constexpr float kLazyRescale = 8.f;           // log2 units the row maximum may grow before O is rescaled
constexpr int kPlanSlots = 2;
constexpr int kPlanReaders = 8 + 2 + kProducerWarps;   // one arrival per softmax warp, per MMA thread, per producer warp

// What the roles need to know about one item.
struct Plan {
  int l, b, h, hq0, has1, gi, q0, T_b;
  int n_tiles;                                // 0: nothing to do (query tile beyond the sequence)
  int nseg, c_lo, uniform, r_lo, r_hi;
  int seg_rho[kMaxSeg], seg_n[kMaxSeg], seg_first[kMaxSeg + 1];
  int tb[kMaxSeg];                            // sequence length at the rounds r_lo .. r_hi - 1 (those that fire inside the query tile)
};

struct Shared {
  uint64_t kv_full[kStages], kv_empty[kStages], s_full[2][2], p_full[2][2], o_done[2][2];
  uint64_t q_full, q_empty, plan_full[kPlanSlots], plan_empty[kPlanSlots], drain[2];
  uint32_t tmem;
  int abort;
  Plan plan[kPlanSlots];
};

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// two floats in one 64-bit register for the packed fp32 instructions (fma / add on both halves at once)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Bounded wait that also gives up as soon as another thread of the CTA has given up.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, Shared* sh, int32_t* dev_status) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  for (uint32_t spins = 0;; ++spins) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((spins & 63u) == 63u) {
      if (*(volatile int*)&sh->abort) return false;
      if (ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
        *(volatile int*)&sh->abort = 1;
        set_dev_status(dev_status, NGC_DEV_TIMEOUT);
        return false;
      }
    }
  }
}
// The same for a whole warp: every lane gets the same answer.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, Shared* sh, int32_t* dev_status) {
  return __all_sync(0xffffffffu, wait_or_abort(bar, parity, sh, dev_status));
}

// Tensor maps of a launch: Q as a 2-D tensor (channel, row over all layers / sequences / heads), box = 64 channels x
// 128 rows; the output over the same rows, box = 32 channels x 32 rows (one warp's chunk).
struct Maps { CUtensorMap q, out; };

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, const void* src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(ptx::smem_u32(src))
               : "memory");
}

// swizzled byte offset of 16-byte piece c (0..15) of key row r inside a K or V tile
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return (uint32_t)((c >> 3) * kKBox + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(ptx::smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(ptx::smem_u32(bar))
               : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
replay_attn_umma_kernel(const __grid_constant__ Maps maps, ReplayAttnParams p, int n_items) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ Shared sh;

  uint8_t* base = (uint8_t*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = base;                                   // [2 heads][32 KB]
  uint8_t* stage = sQ + 2 * kQBytes;                    // [kStages][K 16 KB | V 16 KB]
  uint8_t* sOut = stage + kStages * kStageBytes;        // [8 softmax warps][4 KB]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int pairs = (p.g + 1) >> 1;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&sh.kv_full[s], kProducerLanes); ptx::mbar_init(&sh.kv_empty[s], 2); }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      ptx::mbar_init(&sh.s_full[hh][0], 1); ptx::mbar_init(&sh.s_full[hh][1], 1);
      ptx::mbar_init(&sh.p_full[hh][0], 128); ptx::mbar_init(&sh.p_full[hh][1], 128);
      ptx::mbar_init(&sh.o_done[hh][0], 1); ptx::mbar_init(&sh.o_done[hh][1], 1);
    }
#pragma unroll
    for (int s = 0; s < kPlanSlots; ++s) { ptx::mbar_init(&sh.plan_full[s], 1); ptx::mbar_init(&sh.plan_empty[s], kPlanReaders); }
    ptx::mbar_init(&sh.q_full, 1);
    ptx::mbar_init(&sh.q_empty, 2);
    ptx::mbar_init(&sh.drain[0], 1);
    ptx::mbar_init(&sh.drain[1], 1);
    ptx::fence_barrier_init();
    sh.abort = 0;
    ptx::prefetch_tensormap(&maps.q);
    ptx::prefetch_tensormap(&maps.out);
  }
  if (warp == kMmaWarp) umma::tmem_alloc(&sh.tmem, kTmemCols);
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem = sh.tmem;

  // Every role walks the same items in the same order: item k of this CTA is blockIdx.x + k * gridDim.x and uses plan
  // slot k & 1.  Ring positions and barrier phases follow from running counters that every role keeps for itself:
  // tiles of all items so far -> K/V stage, S buffer and P / O phases of head 0; tiles of the items that have a second
  // head -> those of head 1.

  if (warp == kPlannerWarp) {
    // ------------------------------------------------------------------ planner: item tables, then Q
    int n_q = 0;                                        // items that had tiles (Q loads) so far
    int k = 0;
    for (int it = blockIdx.x; it < n_items; it += gridDim.x, ++k) {
      const int slot = k & 1;
      if (k >= kPlanSlots && !warp_wait(&sh.plan_empty[slot], ((k >> 1) - 1) & 1, &sh, p.dev_status)) break;
      Plan& pl = sh.plan[slot];
      int item = it;
      const int m = item % p.q_tiles; item /= p.q_tiles;
      const int pair = item % pairs; item /= pairs;
      const int h = item % p.Hkv; item /= p.Hkv;
      const int b = item % p.B;
      const int l = item / p.B;
      const int T_b = min(p.lens[b], p.t_max);
      const int q0 = m * kQRows;
      const int hq0 = h * p.g + 2 * pair;
      const int has1 = 2 * pair + 1 < p.g;              // an odd group leaves the last pair half empty
      const int gi = list_of(p.lists, l, h, p.Hkv);
      int n_tiles = 0;
      if (q0 < T_b) {
        const int q_last = min(q0 + kQRows - 1, T_b - 1);
        // rounds fired before the first / last query of the tile: counted by the whole warp (independent loads)
        int n_lo = 0, n_hi = 0;
        for (int r = lane; r < p.n_rounds; r += 32) {
          const int tb = p.total_before[r * p.B + b];
          n_lo += tb <= q0;
          n_hi += tb <= q_last;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          n_lo += __shfl_xor_sync(0xffffffffu, n_lo, o);
          n_hi += __shfl_xor_sync(0xffffffffu, n_hi, o);
        }
        const int r_lo = n_lo;
        int r_hi = n_hi;
        // key sources of the tile: the kept lists of the rounds it straddles (rho = r_lo .. r_hi, from 1), then the contiguous run
        const int rho0 = max(r_lo, 1);
        if (r_hi - rho0 + 1 > kMaxSeg - 1) {            // more rounds inside one query tile than the table holds
          if (lane == 0) set_dev_status(p.dev_status, NGC_DEV_BAD_COUNTS);
          r_hi = rho0 + kMaxSeg - 2;
        }
        for (int rho = rho0 + lane; rho <= r_hi; rho += 32) {
          int n = p.alive_count[((int64_t)(rho - 1) * p.B + b) * p.G + gi];
          if (n < 0 || n > p.kt_max) { set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT); n = 0; }
          pl.seg_n[rho - rho0] = n;                     // provisional: compacted below by lane 0
        }
        for (int r = r_lo + lane; r < r_hi; r += 32) pl.tb[r - r_lo] = p.total_before[r * p.B + b];
        const int c_lo = r_lo >= 1 ? p.total_before[(r_lo - 1) * p.B + b] : 0;
        __syncwarp();
        if (lane == 0) {
          int nseg = 0, first = 0;
          for (int rho = rho0; rho <= r_hi; ++rho) {
            const int n = pl.seg_n[rho - rho0];         // read before the slot can be overwritten (nseg <= rho - rho0)
            if (n > 0) {
              pl.seg_rho[nseg] = rho; pl.seg_n[nseg] = n; pl.seg_first[nseg] = first;
              first += (n + kKeys - 1) / kKeys;
              ++nseg;
            }
          }
          pl.c_lo = c_lo;
          pl.seg_rho[nseg] = -1; pl.seg_n[nseg] = q_last - c_lo + 1; pl.seg_first[nseg] = first;
          first += (q_last - c_lo + kKeys) / kKeys;
          ++nseg;
          pl.seg_first[nseg] = first;
          pl.nseg = nseg;
          pl.uniform = r_lo == r_hi;                    // every query of the tile lies in the same block
          pl.r_lo = r_lo; pl.r_hi = r_hi;
          pl.n_tiles = first;
        }
        __syncwarp();
        n_tiles = pl.n_tiles;
      }
      if (lane == 0) {
        pl.l = l; pl.b = b; pl.h = h; pl.hq0 = hq0; pl.has1 = has1; pl.gi = gi; pl.q0 = q0; pl.T_b = T_b;
        if (n_tiles == 0) pl.n_tiles = 0;
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&sh.plan_full[slot]);
      if (n_tiles == 0) continue;
      // Q tiles of the two heads -> shared memory (rows beyond the sequence: zeros), once the previous item's
      // last S product has read the buffer
      if (n_q >= 1 && !warp_wait(&sh.q_empty, (n_q - 1) & 1, &sh, p.dev_status)) break;
      if (lane == 0) {
        // rows beyond the sequence (or beyond t_max: the next head's rows, zeros past the end of the tensor) only feed
        // the S rows of queries that do not exist and are never written
        const int n_heads = has1 ? 2 : 1;
        ptx::mbar_expect_tx(&sh.q_full, (uint32_t)(n_heads * kQBytes));
        for (int hh = 0; hh < n_heads; ++hh) {
          const int y = (int)((((int64_t)l * p.B + b) * p.Hq + hq0 + hh) * (int64_t)p.t_max + q0);
          tma_load_2d(sQ + hh * kQBytes, &maps.q, 0, y, &sh.q_full);
          tma_load_2d(sQ + hh * kQBytes + kQHalf, &maps.q, 64, y, &sh.q_full);
        }
      }
      __syncwarp();
      ++n_q;
    }
  } else if (warp >= kProducerWarp0) {
    // ------------------------------------------------------------------ producers: cp.async gathers
    const int pw = warp - kProducerWarp0;               // producer warp w gathers key rows 16 w .. 16 w + 15 of a tile
    int issued = 0;                                     // tiles, over all items
    bool ok = true;
    int k = 0;
    for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x, ++k) {
      const int slot = k & 1;
      if (!warp_wait(&sh.plan_full[slot], (k >> 1) & 1, &sh, p.dev_status)) break;
      const Plan& pl = sh.plan[slot];
      const int n_tiles = pl.n_tiles, nseg = pl.nseg, c_lo = pl.c_lo, T_b = pl.T_b, b = pl.b, gi = pl.gi;
      const __nv_bfloat16* k_strip = p.k + ((int64_t)(pl.l * p.Hkv + pl.h) * p.rows_R + p.seq_off[b]) * 128;
      const __nv_bfloat16* v_strip = p.v + ((int64_t)(pl.l * p.Hkv + pl.h) * p.rows_R + p.seq_off[b]) * 128;
      // position of key row 16 pw + (lane & 15) of tile i, one coalesced load per tile, fetched one tile ahead.  A row
      // the tile does not have (beyond the segment's end) is fetched from position 0 of the sequence: live data that
      // the mask gives weight 0 (every byte of a stage comes through cp.async, so the mbarrier hand-over covers it);
      // a kept position outside the sequence is reported and treated the same way.
      int sgi = 0;
      auto tile_pos = [&](int i) {
        while (sgi + 1 < nseg && i >= pl.seg_first[sgi + 1]) ++sgi;
        const int rho = pl.seg_rho[sgi], n = pl.seg_n[sgi];
        const int kidx = (i - pl.seg_first[sgi]) * kKeys + 16 * pw + (lane & 15);
        if (kidx >= n) return 0;
        const int pos = rho >= 1 ? p.alive_pos[(((int64_t)(rho - 1) * p.B + b) * p.G + gi) * p.kt_max + kidx] : c_lo + kidx;
        if (pos >= 0 && pos < T_b) return pos;
        set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT);
        return 0;
      };
      int pos_next = n_tiles > 0 ? tile_pos(0) : 0;
      for (int i = 0; i < n_tiles; ++i) {
        const int s = issued % kStages;
        const int pos_mine = pos_next;
        if (i + 1 < n_tiles) pos_next = tile_pos(i + 1);
        if (issued >= kStages && !warp_wait(&sh.kv_empty[s], ((issued / kStages) - 1) & 1, &sh, p.dev_status)) { ok = false; break; }
        uint8_t* st = stage + s * kStageBytes;
        const int c = lane & 15;
#pragma unroll
        for (int u = 0; u < 8; ++u) {                   // two rows per step, 16 lanes (16-byte pieces) per row
          const int rl = 2 * u + (lane >> 4);
          const int pos = __shfl_sync(0xffffffffu, pos_mine, rl);
          const uint32_t off = tile_off(16 * pw + rl, c);
          ptx::cp_async_cg_16(ptx::smem_u32(st + off), k_strip + (int64_t)pos * 128 + 8 * c);
          ptx::cp_async_cg_16(ptx::smem_u32(st + kKTile + off), v_strip + (int64_t)pos * 128 + 8 * c);
        }
        ptx::cp_async_mbar_arrive_noinc(&sh.kv_full[s]);    // counts as this lane's arrival once its copies have landed
        ++issued;
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&sh.plan_empty[slot]);
    }
    ptx::cp_async_wait_all();
  } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
    // ------------------------------------------------------------------ MMA issue: one thread per head
    // Two issuing threads halve the serial issue path (descriptors, waits, fences, commits) per tile; the tensor
    // pipe takes their instructions as they come.  Both threads release a K/V stage and the Q buffer (two
    // arrivals each); for an item without a second head the thread of head 1 just passes the arrivals on.
    const int hh = warp - kMmaWarp;
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma::instr_desc(kQRows, kKeys, false);
      constexpr uint32_t idesc_o = umma::instr_desc(kQRows, 128, true);
      const uint32_t st_addr = ptx::smem_u32(stage);
      const uint32_t o_tmem = tmem + 256u + 128u * hh;
      // Operand descriptors differ only in their low word (start address / 16): the Q descriptors of the eight
      // 16-channel steps are fixed, those of K and V follow the stage.  High word: stride 1024 bytes between 8-row
      // groups, descriptor version 1, 128-byte swizzle.
      const uint64_t desc_hi = (uint64_t)umma::smem_desc_sw128(0, 0, 1024) & 0xffffffff00000000ull;
      const uint32_t q_lo = ((ptx::smem_u32(sQ) + hh * kQBytes) >> 4) | (1u << 16);      // leading offset 16 bytes (unused with swizzle)
      const uint32_t v_lbo = (uint32_t)(kKBox >> 4) << 16;                                // V: the next 64 channels are one box on
      int t0 = 0, th = 0, n_q = 0;                      // tiles so far (all items / items with this head), items with tiles so far
      int st_cur = 0, ph_cur = 0;                       // stage and phase parity of tile t0
      bool ok = true;
      int k = 0;
      for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x, ++k) {
        const int slot = k & 1;
        if (!wait_or_abort(&sh.plan_full[slot], (k >> 1) & 1, &sh, p.dev_status)) break;
        const int n_tiles = sh.plan[slot].n_tiles;
        const bool mine = hh == 0 || sh.plan[slot].has1;
        ptx::mbar_arrive(&sh.plan_empty[slot]);         // nothing else of the table is needed here
        if (n_tiles == 0) continue;
        ok = wait_or_abort(&sh.q_full, n_q & 1, &sh, p.dev_status);      // (also: the previous use of q_empty is over)
        if (!ok) break;
        if (!mine) {
          // nothing to multiply: hand on this thread's share of the releases, each after the tile has landed (so
          // that the arrival cannot fall into an earlier phase of the stage's barrier)
          ptx::mbar_arrive(&sh.q_empty);
          for (int i = 0; i < n_tiles && ok; ++i) {
            ok = wait_or_abort(&sh.kv_full[st_cur], ph_cur, &sh, p.dev_status);
            if (ok) ptx::mbar_arrive(&sh.kv_empty[st_cur]);
            if (++st_cur == kStages) { st_cur = 0; ph_cur ^= 1; }
          }
          t0 += n_tiles;
          ++n_q;
          continue;
        }
        auto issue_s = [&](int stg, int buf, bool last) {      // S = Q K^T for the tile in stage stg, into S buffer buf
          const uint32_t k_lo = ((st_addr + stg * kStageBytes) >> 4) | (1u << 16);
          const uint32_t d = tmem + (uint32_t)((2 * hh + buf) * kKeys);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint64_t a = desc_hi | (uint64_t)(q_lo + (uint32_t)(((ks >> 2) * kQHalf + (ks & 3) * 32) >> 4));
            const uint64_t bd = desc_hi | (uint64_t)(k_lo + (uint32_t)(((ks >> 2) * kKBox + (ks & 3) * 32) >> 4));
            umma::mma_bf16(d, a, bd, idesc_s, ks > 0);
          }
          umma::commit(&sh.s_full[hh][buf]);
          if (last) umma::commit(&sh.q_empty);          // the item's last product that reads Q
        };
        ok = wait_or_abort(&sh.kv_full[st_cur], ph_cur, &sh, p.dev_status);
        if (!ok) break;
        issue_s(st_cur, th & 1, n_tiles == 1);
        for (int i = 0; i < n_tiles; ++i) {
          int st_nxt = st_cur + 1, ph_nxt = ph_cur;
          if (st_nxt == kStages) { st_nxt = 0; ph_nxt ^= 1; }
          const int tt = th + i;                        // tile count of this head: P sits in S buffer tt & 1, use tt >> 1 of it
          if (i + 1 < n_tiles) {
            ok = wait_or_abort(&sh.kv_full[st_nxt], ph_nxt, &sh, p.dev_status);
            if (!ok) break;
            issue_s(st_nxt, (tt + 1) & 1, i + 2 == n_tiles);   // its buffer held S and P of two tiles ago: that P V product was issued
                                                               // before this one, and the tensor pipe runs them in issue order
          }
          ok = wait_or_abort(&sh.p_full[hh][tt & 1], (tt >> 1) & 1, &sh, p.dev_status);
          if (!ok) break;
          umma::fence_after_sync();                     // P was written with tcgen05.st by the softmax threads
          const uint32_t v_lo = ((st_addr + st_cur * kStageBytes + kKTile) >> 4) | v_lbo;
          const uint32_t p_tmem = tmem + (uint32_t)((2 * hh + (tt & 1)) * kKeys);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)                // 16 keys per step: 8 packed columns of P, two 8-row groups of V
            umma::mma_bf16_a_tmem(o_tmem, p_tmem + 8 * kk, desc_hi | (uint64_t)(v_lo + (uint32_t)((kk * 2048) >> 4)), idesc_o,
                                  (i > 0 || kk > 0) ? 1u : 0u);
          umma::commit(&sh.o_done[hh][tt & 1]);
          umma::commit(&sh.kv_empty[st_cur]);           // this head is done with K and V of the stage
          st_cur = st_nxt; ph_cur = ph_nxt;
        }
        t0 += n_tiles;
        th += n_tiles;
        ++n_q;
      }
      // everything issued has completed before tensor memory is released
      umma::commit(&sh.drain[hh]);
      wait_or_abort(&sh.drain[hh], 0, &sh, p.dev_status);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax: one thread per query row
    const int hh = warp >> 2;
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const uint32_t o_addr = tmem + lane_base + 256u + 128u * hh;
    int tc = 0;                                         // tiles this head has been through, over all items
    bool ok = true;
    int k = 0;
    for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x, ++k) {
      const int slot = k & 1;
      if (!warp_wait(&sh.plan_full[slot], (k >> 1) & 1, &sh, p.dev_status)) break;
      const Plan& pl = sh.plan[slot];
      const int n_tiles = (hh == 0 || pl.has1) ? pl.n_tiles : 0;
      if (n_tiles > 0) {
        const int q0 = pl.q0, T_b = pl.T_b, c_lo = pl.c_lo, nseg = pl.nseg;
        const bool uniform = pl.uniform != 0;
        const int t_q = q0 + row;
        int blk = pl.r_lo, lo_row = c_lo;               // round index of the row's block, its first position
        for (int r = pl.r_lo; r < pl.r_hi; ++r) {       // the rounds that fire inside this query tile
          const int tb = pl.tb[r - pl.r_lo];
          if (tb <= t_q) { blk += 1; lo_row = tb; }
        }
        float m_use = -INFINITY, l_run = 0.f;
        int o_seen = tc - 1;                            // last tile whose P V product is known to be complete (they complete in order)
        int sgi = 0;
        for (int i = 0; i < n_tiles; ++i) {
          const int t = tc + i;
          if (!warp_wait(&sh.s_full[hh][t & 1], (t >> 1) & 1, &sh, p.dev_status)) { ok = false; break; }
          umma::fence_after_sync();
          uint32_t zr[2][32];
          const uint32_t s_addr = tmem + lane_base + (uint32_t)((2 * hh + (t & 1)) * kKeys);
          umma::tmem_ld32(s_addr, zr[0]);
          umma::tmem_ld32(s_addr + 32, zr[1]);
          umma::tmem_ld_wait();
          while (sgi + 1 < nseg && i >= pl.seg_first[sgi + 1]) ++sgi;
          const int rho = pl.seg_rho[sgi], kt = i - pl.seg_first[sgi];
          const int n_here = min(kKeys, pl.seg_n[sgi] - kt * kKeys);
          // a tile needs no mask when every query of the item lies in one block and the tile is a full tile of that
          // block's kept list, or lies entirely before the first query
          const bool need_mask = !uniform || (rho >= 1 ? n_here < kKeys : c_lo + kt * kKeys + kKeys - 1 > q0);
          // raw scores stay as they are; invisible ones become -inf.  The row maximum is taken on the raw values
          // (the scale is positive) with three-input max over four independent chains.
          if (need_mask) {
            // the visible keys of this row are one index range of the tile: the whole kept tile (up to its end) if the
            // row's block follows that round, else nothing; or the causal part of the row's own block
            int jlo, jhi;
            if (rho >= 1) { jlo = blk == rho ? 0 : kKeys; jhi = n_here - 1; }
            else { const int j0 = c_lo + kt * kKeys; jlo = max(lo_row - j0, 0); jhi = t_q - j0; }
            const uint32_t width = jhi >= jlo ? (uint32_t)(jhi - jlo) : 0u;
            if (jhi < jlo) jlo = 2 * kKeys;                                    // nothing visible
#pragma unroll
            for (int half = 0; half < 2; ++half)
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if ((uint32_t)(32 * half + j - jlo) > width) zr[half][j] = 0xff800000u;   // -inf
          }
          float mxc[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int half = 0; half < 2; ++half)
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
#pragma unroll
              for (int c = 0; c < 4; ++c)
                mxc[c] = max3(mxc[c], __uint_as_float(zr[half][j + 2 * c]), __uint_as_float(zr[half][j + 2 * c + 1]));
            }
          const float mx = fmaxf(fmaxf(mxc[0], mxc[1]), fmaxf(mxc[2], mxc[3])) * p.scale_log2;
          // the maximum used for the exponentials follows the true one lazily
          const bool grow = mx > m_use + kLazyRescale;                        // also the first visible key (m_use = -inf)
          const bool rescale = grow && m_use != -INFINITY && i > 0;           // O already holds something for this row
          if (__any_sync(0xffffffffu, rescale)) {
            if (o_seen < t - 1) {
              if (!warp_wait(&sh.o_done[hh][(t - 1) & 1], ((t - 1) >> 1) & 1, &sh, p.dev_status)) { ok = false; break; }
              o_seen = t - 1;
              umma::fence_after_sync();
            }
            const float alpha = rescale ? ptx::ex2_approx(m_use - mx) : 1.f;
            l_run *= alpha;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
              uint32_t o[32];
              umma::tmem_ld32(o_addr + c0, o);
              umma::tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
              umma::tmem_st32(o_addr + c0, o);
            }
            umma::tmem_st_wait();
          }
          if (grow) m_use = mx;
          const float m_eff = m_use == -INFINITY ? 0.f : m_use;               // nothing visible yet: every exponential is 0
          // p = 2^(z * scale - m): one packed fused multiply-add per pair of scores, then the exponentials; the row sum
          // in four independent packed chains
          const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nm2 = pack2(-m_eff, -m_eff);
          uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};
          uint32_t pk[32];
#pragma unroll
          for (int half = 0; half < 2; ++half)
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              float x0, x1;
              unpack2(fma2(pack2(__uint_as_float(zr[half][j]), __uint_as_float(zr[half][j + 1])), sc2, nm2), x0, x1);
              const float p0 = ptx::ex2_approx(x0), p1 = ptx::ex2_approx(x1);
              acc2[(j >> 1) & 3] = add2(acc2[(j >> 1) & 3], pack2(p0, p1));
              pk[16 * half + (j >> 1)] = ptx::pack_bf16x2(p0, p1);
            }
          {
            float s0, s1;
            unpack2(add2(add2(acc2[0], acc2[1]), add2(acc2[2], acc2[3])), s0, s1);
            l_run += s0 + s1;
          }
          // P over the first 32 columns of the S buffer this row was just read from (free: the row is in registers)
          umma::tmem_st32(s_addr, pk);
          umma::tmem_st_wait();
          umma::fence_before_sync();
          ptx::mbar_arrive(&sh.p_full[hh][t & 1]);
        }
        if (!ok) break;
        tc += n_tiles;
        if (!warp_wait(&sh.o_done[hh][(tc - 1) & 1], ((tc - 1) >> 1) & 1, &sh, p.dev_status)) { ok = false; break; }
        umma::fence_after_sync();
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
        // The thread owns a whole output row.  Every 32-column chunk goes through the warp's 4 KB of shared memory (each
        // thread its own row, in the swizzle TMA expects for a box of that row width) and leaves as ONE asynchronous TMA
        // store per warp: the load/store unit, busy with the producers' gathers, is not involved.  A warp whose 32 rows
        // reach beyond the sequence must not write those rows: it stores with ordinary instructions, several lanes per row.
        uint8_t* so = sOut + warp * kOutStage;
        const int t_w0 = q0 + 32 * (warp & 3);                                // query token of this warp's row 0
        const int64_t o_row0 = ((((int64_t)pl.l * p.B + pl.b) * p.Hq + pl.hq0 + hh) * (int64_t)p.t_max + t_w0) * 128;
        const bool whole = t_w0 + 32 <= T_b;
        // The chunk after the current one is already on its way out of tensor memory while this one is scaled,
        // packed and handed to the TMA unit.
        uint32_t ob[2][32];
        umma::tmem_ld32(o_addr, ob[0]);
#pragma unroll
        for (int ci = 0; ci < 4; ++ci) {
          const int c0 = 32 * ci;
          uint32_t (&o)[32] = ob[ci & 1];
          umma::tmem_ld_wait();
          if (ci < 3) umma::tmem_ld32(o_addr + c0 + 32, ob[(ci + 1) & 1]);
          if (lane == 0) ptx::bulk_wait_read<0>();                            // the previous chunk's store has read the staging area
          __syncwarp();
          if (p.out_bf16) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
              *reinterpret_cast<uint4*>(so + lane * 64 + ((c ^ ((lane >> 1) & 3)) << 4)) =
                  make_uint4(ptx::pack_bf16x2(__uint_as_float(o[8 * c]) * inv, __uint_as_float(o[8 * c + 1]) * inv),
                             ptx::pack_bf16x2(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv),
                             ptx::pack_bf16x2(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv),
                             ptx::pack_bf16x2(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv));
          } else {
#pragma unroll
            for (int c = 0; c < 8; ++c)
              *reinterpret_cast<float4*>(so + lane * 128 + ((c ^ (lane & 7)) << 4)) =
                  make_float4(__uint_as_float(o[4 * c]) * inv, __uint_as_float(o[4 * c + 1]) * inv,
                              __uint_as_float(o[4 * c + 2]) * inv, __uint_as_float(o[4 * c + 3]) * inv);
          }
          if (whole) {
            ptx::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&maps.out, c0, (int)(o_row0 >> 7), so);
              ptx::bulk_commit();
            }
          } else if (p.out_bf16) {
            __syncwarp();
#pragma unroll
            for (int u = 0; u < 4; ++u) {                                     // eight rows per store, four lanes per row
              const int r = 8 * u + (lane >> 2), c = lane & 3;
              const uint4 v = *reinterpret_cast<const uint4*>(so + r * 64 + ((c ^ ((r >> 1) & 3)) << 4));
              if (t_w0 + r < T_b)
                *reinterpret_cast<uint4*>((__nv_bfloat16*)p.out + o_row0 + (int64_t)r * 128 + c0 + 8 * c) = v;
            }
          } else {
            __syncwarp();
#pragma unroll
            for (int u = 0; u < 8; ++u) {                                     // four rows per store, eight lanes per row
              const int r = 4 * u + (lane >> 3), c = lane & 7;
              const float4 v = *reinterpret_cast<const float4*>(so + r * 128 + ((c ^ (r & 7)) << 4));
              if (t_w0 + r < T_b)
                *reinterpret_cast<float4*>((float*)p.out + o_row0 + (int64_t)r * 128 + c0 + 4 * c) = v;
            }
          }
        }
        // (the next item's first P V overwrites O only after this thread has published its next P row, which comes
        // after these reads)
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&sh.plan_empty[slot]);
    }
    if (lane == 0) ptx::bulk_wait<0>();                 // this warp's output stores have completed
  }
  // ---- teardown: every role has left its loops; nothing of this CTA is in flight any more
  umma::fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    umma::fence_after_sync();
    umma::tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

int launch_replay_attn_umma(const ReplayAttnParams& p, cudaStream_t stream) {
  const int pairs = (p.g + 1) / 2;
  ReplayAttnParams q = p;
  q.q_tiles = (p.t_max + kQRows - 1) / kQRows;
  const int64_t items = (int64_t)p.L * p.B * p.Hkv * pairs * q.q_tiles;
  if (items > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  // TMA coordinates are 32-bit: queries and outputs are addressed by row over all layers, sequences and heads
  Maps maps;
  if (!make_rows_map(&maps.q, p.q, (int64_t)p.L * p.B * p.Hq * p.t_max, kQRows) ||
      !make_out_map(&maps.out, p.out, p.out_bf16 != 0, (int64_t)p.L * p.B * p.Hq * p.t_max, 32))
    return NGC_ERR_UNSUPPORTED;
  static PerDeviceOnce attr_once;      // the shared-memory opt-in is stored per device
  static int sm_count[kMaxDevices] = {0};
  int dev = -1;
  const int rc = attr_once.run([&] {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_count[cur], cudaDevAttrMultiProcessorCount, cur);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(replay_attn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    return e;
  }, &dev);
  if (rc != NGC_OK) return rc;
  // One CTA per SM by construction (226 KB of shared memory each): a CTA owns all 512 columns of its SM's tensor
  // memory, and walks the items blockIdx.x, blockIdx.x + gridDim.x, ...
  const int grid = (int)(items < sm_count[dev] ? items : sm_count[dev]);
  replay_attn_umma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(maps, q, (int)items);
  return launch_status();
}

}  // namespace ngc
