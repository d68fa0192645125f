// Launch parameters shared by the two device paths of ngc_replay_attn.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ngc {

struct ReplayAttnParams {
  const __nv_bfloat16* k;        // [L][Hkv][R][128]: every token of every sequence, original order
  const __nv_bfloat16* v;
  const int64_t* seq_off;
  const int32_t* lens;           // T_b
  const __nv_bfloat16* q;        // [L][B][Hq][t_max][128]
  const int32_t* alive_pos;      // [n_rounds][B][G][kt_max]
  const int32_t* alive_count;    // [n_rounds][B][G]
  const int32_t* total_before;   // [n_rounds][B]
  void* out;                     // [L][B][Hq][t_max][128]
  int32_t* dev_status;
  int64_t rows_R;
  int L, B, Hq, Hkv, g, t_max, n_rounds, G, kt_max, lists, out_bf16, q_tiles;
  float scale_log2;
};

// The tcgen05 / tensor-memory path (replay_attn_umma.cu): enqueues the kernel, returns an ngc_status.
int launch_replay_attn_umma(const ReplayAttnParams& p, cudaStream_t stream);

}  // namespace ngc
