// ngc_replay_visibility: which original tokens each eviction round left alive (paper Appendix A.3,
// "Reconstructing Replay Attention Masks from Retention Decisions").
//
// The rollout stores, per round and list, the ascending kept units in the coordinates of the
// cache at that round.  The replay pass needs them as ORIGINAL token positions: a query of the
// block that follows round r sees kept_r plus, causally, its own block.  The paper builds dense
// B x T x T masks from this; here the result stays a list per (round, list) -- T entries instead
// of T^2 bits.
//
// One CTA per (sequence, list) walks the rounds in order with the alive set A_r (original
// positions, in cache order) in shared memory: A_r = kept_{r-1} followed by the positions of the
// tokens appended since; kept_r = the entries of A_r at the kept units.  Integer gathers only.
#include "ngc_common.cuh"

namespace ngc {
namespace {

constexpr int kThreads = 256;

struct ReplayParams {
  const int32_t* kept_sorted;    // [R][B][G][k_max]
  const int32_t* budget;         // [R][B]
  const int32_t* alive_before;   // [R][B], or [R][B][G] when per_list
  const int32_t* total_before;   // [R][B]
  int32_t* alive_pos;            // [R][B][G][k_max * block]
  int32_t* alive_count;          // [R][B][G]
  int32_t* dev_status;
  int R, B, G, k_max, block, alive_max, per_list;
};

__global__ void __launch_bounds__(kThreads) replay_visibility_kernel(ReplayParams p) {
  extern __shared__ int32_t s_pos[];              // [2][alive_max]
  __shared__ int s_bad;
  const int b = blockIdx.x / p.G, gi = blockIdx.x - b * p.G;
  const int tid = threadIdx.x;
  int32_t* cur = s_pos;
  int32_t* nxt = s_pos + p.alive_max;
  const int out_stride = p.k_max * p.block;
  int n_prev = 0;                                 // |kept_{r-1}|
  int fail = 0;
  for (int r = 0; r < p.R; ++r) {
    const int64_t li = ((int64_t)r * p.B + b) * p.G + gi;
    int32_t* out = p.alive_pos + li * out_stride;
    if (!fail) {
      const int n_alive = p.per_list ? p.alive_before[li] : p.alive_before[r * p.B + b];
      const int total = p.total_before[r * p.B + b];
      const int K = p.budget[r * p.B + b];
      const int grow = n_alive - n_prev;          // tokens appended since the last round (block_r)
      const int n_units = (n_alive + p.block - 1) / p.block;
      const int32_t* kept = p.kept_sorted + li * p.k_max;
      if (grow < 0 || grow > total || n_alive > p.alive_max || K < 0 || K > p.k_max) {
        fail = NGC_DEV_BAD_COUNTS;
      } else {
        if (tid == 0) s_bad = 0;
        for (int i = tid; i < grow; i += kThreads)
          if (NGC_IN_BOUNDS(p.dev_status, n_prev + i < p.alive_max)) cur[n_prev + i] = total - grow + i;
        __syncthreads();
        int bad = K > n_units ? 1 : 0;
        for (int j = tid; j < K && !bad; j += kThreads) {
          const int u = kept[j];
          const int prev = j > 0 ? kept[j - 1] : -1;
          if (u <= prev || u >= n_units) bad = 1;
        }
        if (bad) atomicOr(&s_bad, 1);
        __syncthreads();
        if (s_bad) {
          fail = NGC_DEV_BAD_KEPT;
        } else {
          // only the last unit of A_r can be short, and if kept it is the last kept unit
          int count = K * p.block;
          if (K > 0 && kept[K - 1] == n_units - 1) count -= n_units * p.block - n_alive;
          for (int i = tid; i < out_stride; i += kThreads) {
            int v = -1;
            if (i < count) {
              const int j = i / p.block;
              const int src = kept[j] * p.block + (i - j * p.block);
              if (NGC_IN_BOUNDS(p.dev_status, src >= 0 && src < n_alive && i < p.alive_max)) {
                v = cur[src];
                nxt[i] = v;
              }
            }
            out[i] = v;
          }
          if (tid == 0) p.alive_count[li] = count;
          __syncthreads();
          int32_t* t = cur; cur = nxt; nxt = t;
          n_prev = count;
        }
      }
      if (fail && tid == 0) set_dev_status(p.dev_status, fail);
    }
    if (fail) {                                   // this round and every later one of the list
      for (int i = tid; i < out_stride; i += kThreads) out[i] = -1;
      if (tid == 0) p.alive_count[li] = -1;
    }
  }
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_replay_visibility(const int32_t* kept_sorted, const int32_t* budget, const int32_t* alive_before,
                                     const int32_t* total_before, int R, int B, int G, int k_max, int block, int alive_max,
                                     int per_list, int32_t* alive_pos, int32_t* alive_count, int32_t* dev_status, ngc_stream stream) {
  NGC_API_RANGE("ngc_replay_visibility");
  using namespace ngc;
  if (!kept_sorted || !budget || !alive_before || !total_before || !alive_pos || !alive_count || R <= 0 || B <= 0 || G <= 0 ||
      k_max <= 0 || block <= 0 || alive_max <= 0)
    return NGC_ERR_INVALID_ARG;
  if ((int64_t)B * G > 0x7fffffffLL) return NGC_ERR_UNSUPPORTED;
  const size_t smem = (size_t)2 * alive_max * 4;
  if (smem > 200 * 1024) return NGC_ERR_UNSUPPORTED;
  if (smem > 48 * 1024)
    NGC_CUDA_TRY(cudaFuncSetAttribute(replay_visibility_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  ReplayParams p;
  p.kept_sorted = kept_sorted; p.budget = budget; p.alive_before = alive_before; p.total_before = total_before;
  p.alive_pos = alive_pos; p.alive_count = alive_count; p.dev_status = dev_status;
  p.R = R; p.B = B; p.G = G; p.k_max = k_max; p.block = block; p.alive_max = alive_max; p.per_list = per_list;
  replay_visibility_kernel<<<(unsigned)(B * G), kThreads, smem, (cudaStream_t)stream>>>(p);
  return launch_status();
}
