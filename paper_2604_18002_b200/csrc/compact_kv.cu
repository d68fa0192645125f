// ngc_compact_kv: physical eviction (paper Section 4.1), in place.
//
// One CTA owns one (layer, KV head, sequence, K-or-V) strip and walks its
// OUTPUT rows in ascending tiles.  Kept units are strictly ascending, so the
// source of output token j is never in front of j: tile i reads rows >= i*T
// only, tile i writes rows [i*T, (i+1)*T).  Hence loads may run ahead of stores
// without ever seeing a moved row, as long as every load of tile i is done
// before the first store of tile i (one __syncthreads per tile).  The leading
// run of tokens that already sit in place is skipped.  HBM-bound: 16-byte
// vector loads/stores, five CTAs per SM, next tile prefetched into registers
// before the current one is stored.  With several lists per sequence and one
// length per sequence, a check kernel runs first: a sequence with a corrupt list,
// or whose lists would keep different token counts, is reported and marked
// (its length entry is complemented for the duration of the call) so that NONE
// of its strips moves; the length kernel behind restores the entry.
// The row width is a template parameter:
// with run-time divisions in the per-vector index arithmetic the kernel was
// issue-bound (ncu: 61 % issue slots busy at 60 % of DRAM throughput).
// (Measured alternatives that were slower on B200: per-row bulk async copies,
// 256 bytes each, are limited by the copy engine's request rate; a cp.async
// gather into a shared-memory ring with one bulk store per 16 KB tile.)
#include "ngc_common.cuh"
#include "ptx.cuh"

namespace ngc {
namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;   // 16-byte vectors per thread per tile

struct CompactParams {
  uint4* k;
  uint4* v;
  const int64_t* seq_off;
  const int32_t* lens;
  const int32_t* kept_sorted;
  const int32_t* budget;
  int32_t* dev_status;
  int64_t plane_vecs;   // R * row_vecs
  int L, B, Hkv, G, lists, block, k_max;
  int row_vecs;         // 16-byte vectors per row
  int lens_lists;       // 0: lens[B]; else == lists: lens[B][G]
};

// Validates one kept list with the whole CTA.  Returns (to every thread) the
// number of kept tokens, or -1 if the list is corrupt.  *first_moved gets the
// first output token whose source differs from its destination.
__device__ int validate_list(const int32_t* kept, int K, int k_max, int len, int block, int* first_moved) {
  __shared__ int s_bad, s_first;
  if (threadIdx.x == 0) { s_bad = 0; s_first = 0x7fffffff; }
  __syncthreads();
  const int n_units = (len + block - 1) / block;
  int bad = (K < 0 || K > k_max || K > n_units) ? 1 : 0;
  int first = 0x7fffffff;
  if (!bad) {
    // eight independent loads per thread in flight: the list may come from HBM
    for (int j0 = threadIdx.x; j0 < K; j0 += 8 * blockDim.x) {
      int u[8], prev[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int j = j0 + e * blockDim.x;
        u[e] = j < K ? kept[j] : 0;
        prev[e] = (j > 0 && j < K) ? kept[j - 1] : -1;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int j = j0 + e * blockDim.x;
        if (j < K) {
          if (u[e] <= prev[e] || u[e] >= n_units) bad = 1;
          if (u[e] != j && j < first) first = j;
        }
      }
    }
  }
  if (bad) atomicOr(&s_bad, 1);
  if (first != 0x7fffffff) atomicMin(&s_first, first);
  __syncthreads();
  bad = s_bad;
  first = s_first;
  __syncthreads();
  if (bad) return -1;
  int tokens = K * block;
  if (K > 0 && kept[K - 1] == n_units - 1) tokens -= n_units * block - len;   // short last unit
  *first_moved = first == 0x7fffffff ? tokens : first * block;
  return tokens;
}

// RV = 16-byte vectors per row (8, 16 or 32: rows of 128, 256 or 512 bytes); compile-time so that
// the row / column split of a thread's vectors costs shifts, not divisions.
template <int RV>
__global__ void __launch_bounds__(kThreads) compact_kernel(CompactParams p) {
  constexpr int kRowsPerPass = kThreads / RV;                 // rows the CTA covers with one vector per thread
  constexpr int kTileRows = kRowsPerPass * kVecPerThread;
  int s = blockIdx.x;
  const int kv = s & 1; s >>= 1;
  const int b = s % p.B; s /= p.B;
  const int h = s % p.Hkv;
  const int l = s / p.Hkv;
  const int gi = list_of(p.lists, l, h, p.Hkv);
  const int len = p.lens[len_index(p.lens_lists, p.L, p.Hkv, b, l, h)];
  if (len < 0) return;          // marked by the check kernel: the sequence stays as it is (already reported)
  const int K = p.budget[b];
  const int32_t* kept = p.kept_sorted + ((int64_t)b * p.G + gi) * p.k_max;

  int first_moved = 0;
  const int tokens = validate_list(kept, K, p.k_max, len, p.block, &first_moved);
  if (tokens < 0) {
    if (threadIdx.x == 0) set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT);
    return;
  }
  const int my_row = threadIdx.x / RV, my_col = threadIdx.x % RV;
  uint4* strip = (kv ? p.v : p.k) + (int64_t)(l * p.Hkv + h) * p.plane_vecs + p.seq_off[b] * RV + my_col;
  const int block = p.block;
#ifdef NGC_DEBUG
  const int64_t cap = p.seq_off[b + 1] - p.seq_off[b];        // rows this sequence owns in the plane
#endif
  uint4 cur[kVecPerThread], nxt[kVecPerThread];
  int src_nxt[kVecPerThread];          // source rows of the tile whose data is fetched next (-1: no such row)

  // The source row of an output row comes from the kept list, which may itself come from HBM (a list per layer and
  // head): the indices are fetched one tile ahead of the rows they address, the rows one tile ahead of their store.
  auto load_sources = [&](int t0, int (&src)[kVecPerThread]) {
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
      const int jt = t0 + u * kRowsPerPass + my_row;
      src[u] = -1;
      if (jt < tokens) {
        if (block == 1) {
          src[u] = __ldg(kept + jt);
        } else {
          const int unit = jt / block;
          src[u] = __ldg(kept + unit) * block + (jt - unit * block);      // < len: validated above
        }
      }
    }
  };
  auto load_tile = [&](int t0, const int (&src)[kVecPerThread], uint4 (&r)[kVecPerThread]) {
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
      const int jt = t0 + u * kRowsPerPass + my_row;
      // a kept row never lies in front of its destination, and always inside the live part of the strip
      if (src[u] >= 0 && NGC_IN_BOUNDS(p.dev_status, src[u] >= jt && src[u] < len && src[u] < cap)) r[u] = __ldcs(strip + (int64_t)src[u] * RV);
    }
  };
  auto store_tile = [&](int t0, const uint4 (&r)[kVecPerThread]) {
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
      const int jt = t0 + u * kRowsPerPass + my_row;
      if (jt < tokens && NGC_IN_BOUNDS(p.dev_status, jt < len && jt < cap)) strip[(int64_t)jt * RV] = r[u];
    }
  };

  int t0 = first_moved;
  if (t0 >= tokens) return;
  load_sources(t0, src_nxt);
  load_tile(t0, src_nxt, cur);
  load_sources(t0 + kTileRows, src_nxt);
  for (; t0 < tokens; t0 += kTileRows) {
    if (t0 + kTileRows < tokens) {
      load_tile(t0 + kTileRows, src_nxt, nxt);
      load_sources(t0 + 2 * kTileRows, src_nxt);
    }
    __syncthreads();            // every load of this tile has completed
    store_tile(t0, cur);
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) cur[u] = nxt[u];
  }
}

// Warp-level check of one kept list (coalesced reads, neighbours through shuffles).
// Returns to every lane the number of kept tokens, or -1 if the list is corrupt.
__device__ int validate_list_warp(const int32_t* kept, int K, int k_max, int len, int block) {
  const int lane = threadIdx.x & 31;
  const int n_units = (len + block - 1) / block;
  if (K < 0 || K > k_max || K > n_units) return -1;
  bool bad = false;
  constexpr int kE = 16;                          // independent loads per lane in flight: a list may come from HBM
  for (int jb = 0; jb < K; jb += 32 * kE) {
    int u[kE];
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      const int j = jb + 32 * e + lane;
      u[e] = j < K ? kept[j] : 0x7fffffff;
    }
    int edge = (lane < kE && jb + 32 * lane > 0 && jb + 32 * lane < K) ? kept[jb + 32 * lane - 1] : -1;
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      const int j = jb + 32 * e + lane;
      int prev = __shfl_up_sync(0xffffffffu, u[e], 1);
      const int first_prev = __shfl_sync(0xffffffffu, edge, e);
      if (lane == 0) prev = first_prev;
      if (j < K && (u[e] <= prev || u[e] >= n_units)) bad = true;
    }
  }
  if (__any_sync(0xffffffffu, bad)) return -1;
  int tokens = K * block;
  if (K > 0 && kept[K - 1] == n_units - 1) tokens -= n_units * block - len;   // short last unit
  return tokens;
}

// Before any strip moves (several lists per sequence, one length per sequence): one CTA per sequence, a
// warp per list, checks every list of the sequence.  If one is corrupt, or the lists would keep different
// token counts (a short last unit that some keep and some evict), the sequence is reported and its length
// entry is replaced by its complement (a negative number) for the rest of the call: the strip kernel
// skips such a sequence entirely and the length kernel restores the entry, so the sequence is left
// exactly as it was.
__global__ void compact_check_kernel(CompactParams p) {
  __shared__ int s_bad, s_min, s_max;
  const int b = blockIdx.x;
  const int K = p.budget[b];
  const int len = p.lens[b];
  if (threadIdx.x == 0) { s_bad = 0; s_min = 0x7fffffff; s_max = -1; }
  __syncthreads();
  const int warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int gi = warp; gi < p.G; gi += n_warps) {
    const int t = len < 0 ? -1 : validate_list_warp(p.kept_sorted + ((int64_t)b * p.G + gi) * p.k_max, K, p.k_max, len, p.block);
    if ((threadIdx.x & 31) == 0) {
      if (t < 0) atomicOr(&s_bad, 1);
      else { atomicMin(&s_min, t); atomicMax(&s_max, t); }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (s_bad) set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT);
    else if (s_min != s_max) set_dev_status(p.dev_status, NGC_DEV_LISTS_DISAGREE);
    if ((s_bad || s_min != s_max) && len >= 0) const_cast<int32_t*>(p.lens)[b] = ~len;
  }
}

// After all strips moved: the lengths become the kept token counts (one CTA per sequence, a warp per
// list; every list is re-validated).  With one length per sequence the lists must agree; with a
// length per list each list gets its own count.  Launched as a programmatic dependent of the strip
// kernel: the lists are checked while the last strips are still moving (neither kernel writes what the
// other reads there), the lengths are written only after the strip kernel has completed.
__global__ void compact_lens_kernel(CompactParams p) {
  __shared__ int s_bad, s_min, s_max;
  const int b = blockIdx.x;
  const int K = p.budget[b];
  const bool per_list = p.lens_lists != 0;          // then lens_lists == lists: every list has its own length
  if (!per_list && p.lens[b] < 0) {                 // marked by the check kernel: put the length back, nothing moved
    __syncthreads();                                // (every thread has read the entry)
    ptx::grid_dep_wait();
    if (threadIdx.x == 0) const_cast<int32_t*>(p.lens)[b] = ~p.lens[b];
    return;
  }
  if (threadIdx.x == 0) { s_bad = 0; s_min = 0x7fffffff; s_max = -1; }
  __syncthreads();
  const int warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int gi = warp; gi < p.G; gi += n_warps) {
    int32_t* len_p = const_cast<int32_t*>(p.lens) + (per_list ? (int64_t)b * p.G + gi : b);
    const int t = validate_list_warp(p.kept_sorted + ((int64_t)b * p.G + gi) * p.k_max, K, p.k_max, *len_p, p.block);
    ptx::grid_dep_wait();                        // every strip has moved (and read its length)
    if ((threadIdx.x & 31) == 0) {
      if (t < 0) atomicOr(&s_bad, 1);            // already reported by the strip kernel
      else if (per_list) *len_p = t;             // lists may keep different token counts (a short last unit)
      else { atomicMin(&s_min, t); atomicMax(&s_max, t); }
    }
  }
  ptx::grid_dep_wait();
  __syncthreads();
  if (threadIdx.x == 0 && !per_list && !s_bad) {
    if (s_min != s_max) set_dev_status(p.dev_status, NGC_DEV_LISTS_DISAGREE);
    else const_cast<int32_t*>(p.lens)[b] = s_min;
  }
}

// ---------------------------------------------------------------- paged caches: eviction edits the page table
//
// One CTA per sequence, a warp per list.  The warp checks its kept list, then rewrites the
// list's page-table row: kept pages first, in kept order, the other pages behind them as
// free pages (relative order kept).  The old row is staged in shared memory; positions come
// from ballots and popcounts.  When every list of the sequence is valid and they agree on the
// kept token count, lens[b] is updated.

struct PageEvictParams {
  int32_t* page_table;     // [B][G][pages_cap]
  int32_t* lens;
  const int32_t* kept_sorted;
  const int32_t* budget;
  int32_t* dev_status;
  int B, G, k_max, page, pages_cap, per_list;
};

__global__ void evict_pages_kernel(PageEvictParams p) {
  extern __shared__ int32_t s_rows[];                  // [n_warps][pages_cap] old table rows
  __shared__ int s_bad, s_min, s_max;
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const int K = p.budget[b];
  if (threadIdx.x == 0) { s_bad = 0; s_min = 0x7fffffff; s_max = -1; }
  __syncthreads();
  int32_t* old_row = s_rows + warp * p.pages_cap;
  for (int gi = warp; gi < p.G; gi += n_warps) {
    int32_t* len_p = p.lens + (p.per_list ? (int64_t)b * p.G + gi : b);
    const int len = *len_p;
    const int n_units = (len + p.page - 1) / p.page;
    const int32_t* kept = p.kept_sorted + ((int64_t)b * p.G + gi) * p.k_max;
    int32_t* row = p.page_table + ((int64_t)b * p.G + gi) * p.pages_cap;
    const int t = n_units <= p.pages_cap ? validate_list_warp(kept, K, p.k_max, len, p.page) : -1;
    if (t < 0) {
      if (lane == 0) { atomicOr(&s_bad, 1); set_dev_status(p.dev_status, NGC_DEV_BAD_KEPT); }
      continue;
    }
    if (lane == 0) {
      if (p.per_list) *len_p = t;                  // every list has its own length
      else { atomicMin(&s_min, t); atomicMax(&s_max, t); }
    }
    for (int j = lane; j < p.pages_cap; j += 32) old_row[j] = row[j];
    __syncwarp();
    // kept pages to the front
    for (int j = lane; j < K; j += 32)
      if (NGC_IN_BOUNDS(p.dev_status, kept[j] >= 0 && kept[j] < p.pages_cap && j < p.pages_cap)) row[j] = old_row[kept[j]];
    // the others behind them: walk the old row 32 entries at a time; an entry is kept iff it
    // appears in the (ascending) kept list, found by binary search
    int out = K;
    for (int j0 = 0; j0 < p.pages_cap; j0 += 32) {
      const int j = j0 + lane;
      bool is_free = false;
      if (j < p.pages_cap) {
        int lo = 0, hi = K;                              // first kept[x] >= j
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (kept[mid] < j) lo = mid + 1; else hi = mid; }
        is_free = !(lo < K && kept[lo] == j);
      }
      const uint32_t m = __ballot_sync(0xffffffffu, is_free);
      if (is_free && NGC_IN_BOUNDS(p.dev_status, out + __popc(m & ((1u << lane) - 1u)) < p.pages_cap))
        row[out + __popc(m & ((1u << lane) - 1u))] = old_row[j];
      out += __popc(m);
    }
    __syncwarp();
  }
  __syncthreads();
  if (threadIdx.x == 0 && !p.per_list && !s_bad) {
    if (s_min != s_max) set_dev_status(p.dev_status, NGC_DEV_LISTS_DISAGREE);
    else p.lens[b] = s_min;
  }
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_compact_kv(ngc_cache* c, const int32_t* kept_sorted, const int32_t* budget, int k_max,
                              int lists, int block, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_compact_kv");
  using namespace ngc;
  if (!valid_cache(c) || !kept_sorted || !budget || k_max <= 0 || block <= 0 || lists < 0 || lists > 2)
    return NGC_ERR_INVALID_ARG;
  if (c->lens_lists != 0 && c->lens_lists != lists) return NGC_ERR_INVALID_ARG;   // a length per eviction list, or one per sequence
  const int row_bytes = c->d * elt_bytes(c->dtype);
  CompactParams p;
  p.k = (uint4*)c->k;
  p.v = (uint4*)c->v;
  p.seq_off = c->seq_off;
  p.lens = c->lens;
  p.kept_sorted = kept_sorted;
  p.budget = budget;
  p.dev_status = dev_status;
  p.row_vecs = row_bytes / 16;
  p.plane_vecs = c->rows * p.row_vecs;
  p.L = c->L; p.B = c->B; p.Hkv = c->Hkv;
  p.G = lists_G(lists, c->L, c->Hkv);
  p.lists = lists; p.block = block; p.k_max = k_max; p.lens_lists = c->lens_lists;
  const int64_t strips = (int64_t)c->L * c->Hkv * c->B * 2;
  if (strips > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  if ((((uintptr_t)c->k | (uintptr_t)c->v) & 15) != 0) return NGC_ERR_INVALID_ARG;      // rows move as 16-byte vectors
  if (p.row_vecs != 8 && p.row_vecs != 16 && p.row_vecs != 32) return NGC_ERR_UNSUPPORTED;
  const int lens_threads = p.G > 4 ? 1024 : 128;
  if (p.G > 1 && p.lens_lists == 0) {
    // the strips of a sequence must move together or not at all
    compact_check_kernel<<<c->B, lens_threads, 0, (cudaStream_t)stream>>>(p);
    const int rc0 = launch_status();
    if (rc0 != NGC_OK) return rc0;
  }
  if (p.row_vecs == 8) compact_kernel<8><<<(unsigned)strips, kThreads, 0, (cudaStream_t)stream>>>(p);
  else if (p.row_vecs == 16) compact_kernel<16><<<(unsigned)strips, kThreads, 0, (cudaStream_t)stream>>>(p);
  else compact_kernel<32><<<(unsigned)strips, kThreads, 0, (cudaStream_t)stream>>>(p);
  int rc = launch_status();
  if (rc != NGC_OK) return rc;
  NGC_CUDA_TRY(launch_pdl(compact_lens_kernel, dim3((unsigned)c->B), dim3(lens_threads), 0, (cudaStream_t)stream, p));
  return launch_status();
}

extern "C" int ngc_evict_pages(ngc_paged_cache* c, const int32_t* kept_sorted, const int32_t* budget, int k_max,
                               int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_evict_pages");
  using namespace ngc;
  if (!c || !c->page_table || !c->lens || !kept_sorted || !budget || k_max <= 0 || c->B <= 0 || c->L <= 0 || c->Hkv <= 0 ||
      c->pages_cap <= 0 || c->page <= 0 || c->lists < 0 || c->lists > 2)
    return NGC_ERR_INVALID_ARG;
  PageEvictParams p;
  p.page_table = c->page_table; p.lens = c->lens; p.kept_sorted = kept_sorted; p.budget = budget; p.dev_status = dev_status;
  p.B = c->B; p.G = lists_G(c->lists, c->L, c->Hkv); p.k_max = k_max; p.page = c->page; p.pages_cap = c->pages_cap;
  p.per_list = c->lens_per_list != 0;
  const int threads = p.G > 4 ? 256 : 32 * (p.G < 1 ? 1 : p.G);
  const size_t smem = (size_t)(threads / 32) * c->pages_cap * 4;
  if (smem > 96 * 1024) return NGC_ERR_UNSUPPORTED;
  if (smem > 48 * 1024)
    NGC_CUDA_TRY(cudaFuncSetAttribute(evict_pages_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  evict_pages_kernel<<<c->B, threads, smem, (cudaStream_t)stream>>>(p);
  return launch_status();
}
