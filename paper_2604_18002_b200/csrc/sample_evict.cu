// ngc_sample_evict: Gumbel-top-k draw of the keep set (paper Section 4.3).
//
// One CTA per list.  The order "larger perturbed key first, equal keys ->
// smaller index first" is realised on integers: the order-preserving 32-bit
// image of the fp32 key, sorted descending by a STABLE sort of the candidates
// taken in index order.
//  * Lists of up to kSampleSmemMaxUnits candidates: least-significant-digit
//    radix sort in shared memory, seven passes of 5 bits.  Each thread owns a
//    run of consecutive candidates and a private counter per digit; a CTA-wide
//    prefix scan over (digit, thread) turns the counts into stable output
//    offsets, and the thread walks its run again scattering 16-bit candidate
//    indices to their ranks.  No atomics.
//  * Longer lists: 64-bit composite keys (image, inverted index) ordered by a
//    bitonic network in the caller's workspace.
// The kept prefix is then marked in a bitmap whose prefix popcounts place the
// ascending kept list.  Integer work throughout; results do not depend on the
// launch shape.
//
// This translation unit must be compiled WITHOUT fast-math: the Gumbel
// transform is a fixed sequence of correctly rounded fp32 operations.
#include "ngc_common.cuh"
#include "ngc_plan.h"

namespace ngc {
namespace {

// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3") ----
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint2 key) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, ctr.x), lo0 = 0xD2511F53u * ctr.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, ctr.z), lo1 = 0xCD9E8D57u * ctr.z;
    ctr = make_uint4(hi1 ^ ctr.y ^ key.x, lo1, hi0 ^ ctr.w ^ key.y, lo0);
    key.x += 0x9E3779B9u;
    key.y += 0xBB67AE85u;
  }
  return ctr;
}

// Natural logarithm of a positive normal float by a fixed recipe: range
// reduction to m in [sqrt(1/2), sqrt(2)), then log m = 2 atanh((m-1)/(m+1))
// with a degree-4 polynomial in z^2.  Only IEEE round-to-nearest add, mul,
// div and fma, so every machine produces the same bits.
__device__ __forceinline__ float det_log(float x) {
  const uint32_t bits = __float_as_uint(x);
  int e = (int)(bits >> 23) - 127;
  float m = __uint_as_float((bits & 0x007FFFFFu) | 0x3F800000u);
  if (m >= 1.41421354f) { m = __fmul_rn(m, 0.5f); e += 1; }
  const float z = __fdiv_rn(__fsub_rn(m, 1.0f), __fadd_rn(m, 1.0f));
  const float w = __fmul_rn(z, z);
  float p = 2.0f / 9.0f;
  p = __fmaf_rn(p, w, 2.0f / 7.0f);
  p = __fmaf_rn(p, w, 2.0f / 5.0f);
  p = __fmaf_rn(p, w, 2.0f / 3.0f);
  p = __fmaf_rn(p, w, 2.0f);
  const float r = __fmul_rn(z, p);
  return __fmaf_rn((float)e, 0.693147180559945f, r);
}

__device__ __forceinline__ float gumbel_from_word(uint32_t x) {
  const float u = __fmul_rn((float)(2u * (x >> 9) + 1u), 5.9604644775390625e-08f);   // odd multiple of 2^-24
  return -det_log(-det_log(u));
}

// Order-preserving map float -> uint32 (larger float, larger integer; -0 == +0 upstream).
__device__ __forceinline__ uint32_t float_image(float f) {
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct SampleParams {
  const float* logits;
  const int32_t* n;
  const int32_t* n_protect;
  const int32_t* budget;
  int32_t* kept_order;
  int32_t* kept_sorted;
  uint8_t* keep_mask;
  unsigned long long* ws_keys;   // [lists][pad_max] when sorting in global memory
  int32_t* dev_status;
  uint64_t seed, round;
  uint32_t list_base;
  int B, G, n_max, k_max, greedy;
  int pad_max;                   // power of two >= n_max
};

// kRadix: shared-memory radix sort (n_max <= kSampleSmemMaxUnits); otherwise bitonic sort of
// 64-bit keys in the workspace.
template <bool kRadix>
__global__ void sample_kernel(SampleParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_flag;
  __shared__ int s_warp_tot[32];
  __shared__ int s_sel[2][32];
  __shared__ int s_carry;

  const int li = blockIdx.x;
  const int b = li / p.G;
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, n_warps = nthr >> 5;
  const int n = p.n[b];
  const int P = p.n_protect ? p.n_protect[b] : 0;
  const int K = p.budget[b];
  const float* s = p.logits + (int64_t)li * p.n_max;
  int32_t* ko = p.kept_order + (int64_t)li * p.k_max;
  int32_t* ks = p.kept_sorted + (int64_t)li * p.k_max;
  uint8_t* km = p.keep_mask ? p.keep_mask + (int64_t)li * p.n_max : nullptr;

  // shared-memory layout
  uint32_t* img = nullptr;             // [n_max] key images (radix)
  uint16_t* idx_a = nullptr;           // [n_max] candidate order, ping
  uint16_t* idx_b = nullptr;           // [n_max] pong
  uint16_t* hist = nullptr;            // [32 digits][threads] private digit counts, then output offsets (padded)
  uint8_t* dig = nullptr;              // [n_max] digit of the candidate at each position of the order, kept from the counting walk
  unsigned long long* keys = nullptr;  // composite keys (bitonic)
  uint32_t* bitmap;
  if (kRadix) {
    const int n_al = (p.n_max + 7) & ~7;
    const int n_slots = max(p.pad_max, nthr) + 64;     // order arrays: a run per thread, rows of nthr + 2 entries
    img = reinterpret_cast<uint32_t*>(smem_raw);
    idx_a = reinterpret_cast<uint16_t*>(smem_raw + (size_t)n_al * 4);
    idx_b = idx_a + n_slots;
    hist = idx_b + n_slots;
    bitmap = reinterpret_cast<uint32_t*>(hist + 34 * nthr);
    dig = reinterpret_cast<uint8_t*>(bitmap + ((p.n_max + 31) >> 5));
  } else {
    keys = p.ws_keys + (int64_t)li * p.pad_max;
    bitmap = reinterpret_cast<uint32_t*>(smem_raw);
  }

  if (tid == 0) s_flag = 0;
  __syncthreads();
  const bool counts_ok = P >= 0 && P <= K && K <= n && n <= p.n_max && K <= p.k_max;
  const int n_cand = counts_ok ? n - P : 0;
  const int Kp = counts_ok ? K - P : 0;
  int pad = 1;
  while (pad < n_cand) pad <<= 1;

  // ---- perturbed keys: one Philox call serves units 4q .. 4q+3 ----
  if (counts_ok) {
    const uint2 key = make_uint2((uint32_t)p.seed, (uint32_t)(p.seed >> 32));
    const uint32_t list_id = p.list_base + (uint32_t)li;
    int nan_seen = 0;
    for (int q = (P >> 2) + tid; q <= ((n - 1) >> 2) && n > 0; q += nthr) {
      uint32_t w[4] = {0, 0, 0, 0};
      if (!p.greedy) {
        const uint4 r = philox4x32_10(make_uint4((uint32_t)q, list_id, (uint32_t)p.round, (uint32_t)(p.round >> 32)), key);
        w[0] = r.x; w[1] = r.y; w[2] = r.z; w[3] = r.w;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int i = 4 * q + j;
        if (i >= P && i < n) {
          const float si = s[i];
          if (si != si) nan_seen = 1;
          float kf = p.greedy ? si : __fadd_rn(si, gumbel_from_word(w[j]));
          kf = __fadd_rn(kf, 0.0f);                       // -0 -> +0
          if (kRadix) {
            img[i - P] = float_image(kf);
          } else {
            keys[i - P] = ((unsigned long long)float_image(kf) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
          }
        }
      }
    }
    if (!kRadix)
      for (int i = n_cand + tid; i < pad; i += nthr) keys[i] = 0ull;   // below every real key
    if (nan_seen) atomicOr(&s_flag, 1);
  }
  __syncthreads();
  const bool ok = counts_ok && s_flag == 0;
  if (!ok) {
    if (tid == 0) set_dev_status(p.dev_status, counts_ok ? NGC_DEV_NAN_LOGIT : NGC_DEV_BAD_COUNTS);
    for (int j = tid; j < p.k_max; j += nthr) { ko[j] = -1; ks[j] = -1; }
    if (km) for (int i = tid; i < p.n_max; i += nthr) km[i] = 0;
    return;
  }

  int order_per = 1;                           // how the sorted order is laid out (radix path)
  uint32_t order_inv = 0;
  if (kRadix) {
    // ---- stable LSD radix sort of the candidate order, descending image: 7 passes of 5 bits ----
    // Thread t owns the consecutive candidates [t*per, (t+1)*per) and a private counter per digit,
    // cnt[digit][t]; in (digit, thread) order the counters' prefix sums are the stable output
    // offsets.  No atomics, no inter-thread traffic inside the counting and scattering walks.
    // Thread t owns the `per` consecutive positions [t*per, (t+1)*per) of the order; position i is
    // STORED at (i % per) * (nthr + 2) + i / per, so that the lanes of a warp walking their runs in step
    // touch consecutive shared-memory words, and consecutive positions (survivors laid out in order, the
    // ranks read at the end) fall into consecutive banks: row stride nthr + 2 entries = one bank more per row.
    // (The division is a multiplication by ceil(2^32 / per).)
    uint16_t* src = idx_a;
    uint16_t* dst = idx_b;
    uint32_t* cnt_words = reinterpret_cast<uint32_t*>(hist);
    int n_sort = n_cand;                 // candidates that take part in the sort
    uint32_t img_base = 0;               // the sort runs on img - img_base ...
    int n_bits = 32;                     // ... whose values need this many bits
    // Long lists of which at most three quarters are drawn: only candidates that can be drawn are sorted.  An
    // image at or below the Kp-th largest is found bit by bit (counting rounds over values held in registers) and
    // the search stops as soon as at most Kp + Kp / 16 candidates lie at or above it: the few extra candidates cost
    // less in the sort than the remaining rounds would.  The survivors are laid out in index order, so the stable
    // sort below treats equal keys exactly as a sort of the whole list would, and the sort keys are taken relative
    // to that image, which shortens them.
    const bool preselect = nthr == 1024 && n_cand > 8192 && Kp > 0 && 4 * (int64_t)Kp <= 3 * (int64_t)n_cand;
    if (preselect) {
      uint32_t v[16];                    // candidates tid, tid + 1024, ...: images (0 = no such candidate; real images are > 0)
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int i = tid + (k << 10);
        v[k] = i < n_cand ? img[i] : 0u;
      }
      uint32_t piv = 0, mx = 0;
#pragma unroll
      for (int k = 0; k < 16; ++k) mx = max(mx, v[k]);
      mx = __reduce_max_sync(0xffffffffu, mx);
      if (lane == 0) s_warp_tot[warp] = (int)mx;
      __syncthreads();
      mx = __reduce_max_sync(0xffffffffu, (uint32_t)s_warp_tot[lane]);
      int cnt_piv = n_cand;
      for (int bit = 31; bit >= 0; --bit) {
        const uint32_t tr = piv | (1u << bit);
        int c = 0;
#pragma unroll
        for (int k = 0; k < 16; ++k) c += v[k] >= tr ? 1 : 0;
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0) s_sel[bit & 1][warp] = c;
        __syncthreads();                 // (the other half of s_sel is rewritten only after the next barrier)
        const int tot = __reduce_add_sync(0xffffffffu, s_sel[bit & 1][lane]);
        if (tot >= Kp) { piv = tr; cnt_piv = tot; }
        if (cnt_piv <= Kp + (Kp >> 4)) break;            // close enough: a few more candidates than needed go into the sort
      }
      // positions of the surviving candidates in index order: index = 1024 k + 32 warp + lane
      int* s_cnt = reinterpret_cast<int*>(cnt_words);          // [16][32 warps]; free until the sort starts
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const uint32_t bal = __ballot_sync(0xffffffffu, v[k] >= piv);
        if (lane == 0) s_cnt[k * 32 + warp] = __popc(bal);
      }
      __syncthreads();
      {
        const int x = tid < 512 ? s_cnt[tid] : 0;
        int incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp_tot[warp] = incl;
        __syncthreads();
        int before = 0, total = 0;
        for (int w2 = 0; w2 < 16; ++w2) { const int t = s_warp_tot[w2]; total += t; if (w2 < warp) before += t; }
        if (tid < 512) s_cnt[tid] = before + incl - x;
        n_sort = total;
        __syncthreads();
      }
      img_base = piv;
      n_bits = 32 - __clz(mx - piv);                           // 0: every survivor has the same key
    }
    const int per = max(1, (n_sort + nthr - 1) / nthr);
    const uint32_t per_inv = per > 1 ? 0xFFFFFFFFu / (uint32_t)per + 1u : 0u;
    auto slot = [&](uint32_t pos) {
      const uint32_t t = per > 1 ? __umulhi(pos, per_inv) : pos;
      return (pos - t * (uint32_t)per) * (uint32_t)(nthr + 2) + t;
    };
    if (preselect) {
      const int* s_cnt = reinterpret_cast<const int*>(cnt_words);
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int i = tid + (k << 10);
        const bool keep = i < n_cand && img[i] >= img_base;
        const uint32_t bal = __ballot_sync(0xffffffffu, keep);
        if (keep) {
          const int pos = s_cnt[k * 32 + warp] + __popc(bal & ((1u << lane) - 1u));
          if (NGC_IN_BOUNDS(p.dev_status, pos >= 0 && pos < n_sort)) src[slot((uint32_t)pos)] = (uint16_t)i;
        }
      }
      __syncthreads();                   // s_cnt is read before the counters are cleared
    } else {
      for (int k = 0; k < per; ++k) {
        const int i = tid * per + k;
        if (i < n_cand) src[k * (nthr + 2) + tid] = (uint16_t)i;
      }
    }
    // counter x = digit * nthr + thread sits at cnt[x + 2 * (x >> 5)]: one pad word per 32 counters, so that
    // the 32 consecutive counters a thread scans start in a different bank for every lane
    for (int shift = 0; shift < n_bits && Kp > 0; shift += 5) {
      for (int i = tid; i < 17 * nthr; i += nthr) cnt_words[i] = 0u;
      __syncthreads();
      for (int k = 0; k < per && tid * per + k < n_sort; ++k) {
        const uint32_t d = 31u - (((img[src[k * (nthr + 2) + tid]] - img_base) >> shift) & 31u);
        dig[k * nthr + tid] = (uint8_t)d;                       // the scattering walk below needs no second gather
        const uint32_t x = d * nthr + tid;
        hist[x + 2 * (x >> 5)] += 1;
      }
      __syncthreads();
      {
        uint32_t* mine = cnt_words + 17 * tid;          // counters 32*tid .. 32*tid + 31 of the scan order
        uint32_t wv[16];
        int sum = 0;
#pragma unroll
        for (int e = 0; e < 16; ++e) { wv[e] = mine[e]; sum += (int)(wv[e] & 0xFFFFu) + (int)(wv[e] >> 16); }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp_tot[warp] = incl;
        __syncthreads();
        int run = incl - sum;
        {
          // counters in front of this warp's: a scan over the warp totals (one per lane) instead of a serial walk
          const int wt = lane < n_warps ? s_warp_tot[lane] : 0;
          int wincl = wt;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wincl, o);
            if (lane >= o) wincl += t;
          }
          run += __shfl_sync(0xffffffffu, wincl - wt, warp);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int c0 = (int)(wv[e] & 0xFFFFu), c1 = (int)(wv[e] >> 16);
          mine[e] = (uint32_t)run | ((uint32_t)(run + c0) << 16);
          run += c0 + c1;
        }
      }
      __syncthreads();
      for (int k = 0; k < per && tid * per + k < n_sort; ++k) {
        const uint16_t cand = src[k * (nthr + 2) + tid];
        const uint32_t d = dig[k * nthr + tid];
        const uint32_t x = d * nthr + tid;
        const uint32_t pos = hist[x + 2 * (x >> 5)]++;
        if (NGC_IN_BOUNDS(p.dev_status, pos < (uint32_t)n_sort)) dst[slot(pos)] = cand;
      }
      __syncthreads();
      uint16_t* t = src; src = dst; dst = t;
    }
    idx_a = src;        // the sorted order
    order_per = per; order_inv = per_inv;
  } else {
    // ---- bitonic sort, descending ----
    for (int k = 2; k <= pad; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < (pad >> 1); t += nthr) {
          const int i = 2 * t - (t & (j - 1));
          const int l = i + j;
          const unsigned long long x = keys[i], y = keys[l];
          const bool desc = (i & k) == 0;
          if ((x < y) == desc) { keys[i] = y; keys[l] = x; }
        }
        __syncthreads();
      }
    }
  }

  // ---- sigma: the drawn units in descending key order; bitmap of kept units ----
  const int n_words = (n + 31) >> 5;
  for (int wd = tid; wd < n_words; wd += nthr) {
    // protected prefix [0, P)
    const int lo = wd << 5;
    uint32_t m = 0;
    if (P >= lo + 32) m = 0xFFFFFFFFu;
    else if (P > lo) m = (1u << (P - lo)) - 1u;
    bitmap[wd] = m;
  }
  __syncthreads();
  for (int j = tid; j < p.k_max; j += nthr) {
    int idx = -1;
    if (j < Kp) {
      const uint32_t jt = order_per > 1 ? __umulhi((uint32_t)j, order_inv) : (uint32_t)j;
      idx = kRadix ? P + (int)idx_a[((uint32_t)j - jt * (uint32_t)order_per) * (uint32_t)(nthr + 2) + jt]
                   : (int)(0xFFFFFFFFu - (uint32_t)(keys[j] & 0xFFFFFFFFull));
      if (NGC_IN_BOUNDS(p.dev_status, idx >= P && idx < n)) atomicOr(&bitmap[idx >> 5], 1u << (idx & 31));
      else idx = -1;
    }
    ko[j] = idx;
  }
  __syncthreads();

  // ---- ascending kept list from the prefix popcounts of the bitmap ----
  // (radix path: assembled in shared memory over the order arrays, which are dead by now, and written out in one
  // coalesced sweep; a thread's own run of up to 32 entries would otherwise go out as 32 strided stores)
  uint16_t* ks_stage = kRadix ? idx_b : nullptr;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < n_words; base += nthr) {
    const int wd = base + tid;
    const uint32_t m = wd < n_words ? bitmap[wd] : 0u;
    const int cnt = __popc(m);
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp_tot[warp] = incl;
    __syncthreads();
    int warp_off = 0;
    for (int w2 = 0; w2 < warp; ++w2) warp_off += s_warp_tot[w2];
    int pos = s_carry + warp_off + incl - cnt;
    uint32_t mm = m;
    while (mm) {
      const int bit = __ffs(mm) - 1;
      mm &= mm - 1;
      if (NGC_IN_BOUNDS(p.dev_status, pos >= 0 && pos < p.k_max)) {
        if (kRadix) ks_stage[pos] = (uint16_t)((wd << 5) + bit);
        else ks[pos] = (wd << 5) + bit;
      }
      ++pos;
    }
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w2 = 0; w2 < n_warps; ++w2) tot += s_warp_tot[w2];
      s_carry += tot;
    }
    __syncthreads();
  }
  if (kRadix)
    for (int j = tid; j < K && j < p.k_max; j += nthr) ks[j] = (int)ks_stage[j];
  for (int j = K + tid; j < p.k_max; j += nthr) ks[j] = -1;
  if (km) {
    for (int i = tid; i < p.n_max; i += nthr)
      km[i] = (i < n && ((bitmap[i >> 5] >> (i & 31)) & 1u)) ? 1 : 0;
  }
}

// ---------------------------------------------------------------- lists of at most 32 units
//
// The paper's own lists are this small (block-level eviction: 16-22 units, Section 5.1).  A warp
// takes a list, a lane a unit: the rank of a candidate is the number of candidates with a larger
// composite key, counted over 32 shuffles; ballots give the mask and the ascending list.

constexpr int kTinyWarps = 8;

__global__ void __launch_bounds__(kTinyWarps * 32) sample_tiny_kernel(SampleParams p, int n_lists) {
  const int lane = threadIdx.x & 31;
  const int li = blockIdx.x * kTinyWarps + (threadIdx.x >> 5);
  if (li >= n_lists) return;
  const int b = li / p.G;
  const int n = p.n[b];
  const int P = p.n_protect ? p.n_protect[b] : 0;
  const int K = p.budget[b];
  const float* s = p.logits + (int64_t)li * p.n_max;
  int32_t* ko = p.kept_order + (int64_t)li * p.k_max;
  int32_t* ks = p.kept_sorted + (int64_t)li * p.k_max;
  uint8_t* km = p.keep_mask ? p.keep_mask + (int64_t)li * p.n_max : nullptr;

  const bool counts_ok = P >= 0 && P <= K && K <= n && n <= p.n_max && K <= p.k_max;
  const bool cand = counts_ok && lane >= P && lane < n;
  const float si = cand ? s[lane] : 0.f;
  const bool nan_seen = __any_sync(0xffffffffu, cand && si != si);
  if (!counts_ok || nan_seen) {
    if (lane == 0) set_dev_status(p.dev_status, counts_ok ? NGC_DEV_NAN_LOGIT : NGC_DEV_BAD_COUNTS);
    for (int j = lane; j < p.k_max; j += 32) { ko[j] = -1; ks[j] = -1; }
    if (km && lane < p.n_max) km[lane] = 0;
    return;
  }
  const int Kp = K - P;
  // perturbed key of this lane's unit (one Philox call serves units 4q .. 4q+3)
  unsigned long long key = 0ull;                     // below every candidate
  if (cand) {
    float kf = si;
    if (!p.greedy) {
      const uint4 r = philox4x32_10(make_uint4((uint32_t)(lane >> 2), p.list_base + (uint32_t)li, (uint32_t)p.round,
                                               (uint32_t)(p.round >> 32)),
                                    make_uint2((uint32_t)p.seed, (uint32_t)(p.seed >> 32)));
      const uint32_t w = (lane & 3) == 0 ? r.x : ((lane & 3) == 1 ? r.y : ((lane & 3) == 2 ? r.z : r.w));
      kf = __fadd_rn(si, gumbel_from_word(w));
    }
    kf = __fadd_rn(kf, 0.0f);                        // -0 -> +0
    key = ((unsigned long long)float_image(kf) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)lane);
  }
  int rank = 0;                                      // candidates in front of this one
#pragma unroll
  for (int j = 0; j < 32; ++j) rank += __shfl_sync(0xffffffffu, key, j) > key ? 1 : 0;
  const bool drawn = cand && rank < Kp;
  const bool kept = drawn || (lane < P);
  if (drawn && NGC_IN_BOUNDS(p.dev_status, rank < p.k_max)) ko[rank] = lane;
  for (int j = Kp + lane; j < p.k_max; j += 32) ko[j] = -1;
  const uint32_t mask = __ballot_sync(0xffffffffu, kept);
  if (kept && NGC_IN_BOUNDS(p.dev_status, __popc(mask & ((1u << lane) - 1u)) < p.k_max)) ks[__popc(mask & ((1u << lane) - 1u))] = lane;
  for (int j = K + lane; j < p.k_max; j += 32) ks[j] = -1;
  if (km && lane < p.n_max) km[lane] = kept ? 1 : 0;
}

inline int pow2_at_least(int x) {
  int p = 1;
  while (p < x) p <<= 1;
  return p;
}

}  // namespace

size_t sample_workspace_bytes(int B, int G, int n_max) {
  if (n_max <= kSampleSmemMaxUnits) return 0;
  return align256((size_t)B * G * pow2_at_least(n_max) * 8);
}

}  // namespace ngc

extern "C" int ngc_sample_evict(const float* logits, const int32_t* n, const int32_t* n_protect,
                                const int32_t* budget, int B, int G, int n_max, int k_max,
                                uint64_t seed, uint64_t round, uint32_t list_base, int greedy,
                                int32_t* kept_order, int32_t* kept_sorted, uint8_t* keep_mask,
                                void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_sample_evict");
  using namespace ngc;
  if (!logits || !n || !budget || !kept_order || !kept_sorted || B <= 0 || G <= 0 || n_max <= 0 || k_max <= 0)
    return NGC_ERR_INVALID_ARG;
  if ((int64_t)B * G > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  SampleParams p;
  p.logits = logits; p.n = n; p.n_protect = n_protect; p.budget = budget;
  p.kept_order = kept_order; p.kept_sorted = kept_sorted; p.keep_mask = keep_mask;
  p.dev_status = dev_status; p.seed = seed; p.round = round; p.list_base = list_base;
  p.B = B; p.G = G; p.n_max = n_max; p.k_max = k_max; p.greedy = greedy;
  p.pad_max = pow2_at_least(n_max);
  p.ws_keys = nullptr;
  const size_t bitmap_bytes = (size_t)((n_max + 31) / 32) * 4;
  int threads = p.pad_max >= 2048 ? 1024 : (p.pad_max >= 512 ? 256 : 64);
  const unsigned grid = (unsigned)(B * G);
  if (n_max <= 32) {
    sample_tiny_kernel<<<(grid + kTinyWarps - 1) / kTinyWarps, kTinyWarps * 32, 0, (cudaStream_t)stream>>>(p, (int)grid);
  } else if (n_max <= kSampleSmemMaxUnits) {
    const size_t n_al = (size_t)((n_max + 7) & ~7);
    const size_t n_slots = (size_t)(p.pad_max > threads ? p.pad_max : threads) + 64;
    const size_t smem = n_al * 4 + 2 * n_slots * 2 + (size_t)34 * threads * 2 + bitmap_bytes + n_slots;
    if (smem > 48 * 1024)
      NGC_CUDA_TRY(cudaFuncSetAttribute(sample_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    sample_kernel<true><<<grid, threads, smem, (cudaStream_t)stream>>>(p);
  } else {
    const size_t need = sample_workspace_bytes(B, G, n_max);
    if (!ws || ws_bytes < need) return NGC_ERR_WORKSPACE;
    if (bitmap_bytes > 200 * 1024) return NGC_ERR_UNSUPPORTED;
    p.ws_keys = (unsigned long long*)ws;
    if (bitmap_bytes > 48 * 1024)
      NGC_CUDA_TRY(cudaFuncSetAttribute(sample_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bitmap_bytes));
    sample_kernel<false><<<grid, threads, bitmap_bytes, (cudaStream_t)stream>>>(p);
  }
  return launch_status();
}
