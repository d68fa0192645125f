/*
 * CPU oracle for the Neural Garbage Collection hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, sequential restatement of
 * what the paper defines (Sections 4.1-4.3), written to be checked against the
 * paper by eye.  It shares no source, header, table or helper with the CUDA
 * library and must never be called from the product path: only the test
 * suite, the smoke check and the CPU-baseline leg of the benchmark may load it.
 *
 * All pointers are HOST pointers.  Cache layout (same meaning as the CUDA
 * library, restated here independently):
 *   k, v     : [L][Hkv][R][d] elements, R = seq_off[B] rows per (layer, head) plane
 *   seq_off  : [B+1] int64, first row of sequence b inside a plane
 *   lens     : [B] int32, number of alive tokens of sequence b
 *   dtype    : 0 = IEEE fp32, 1 = bfloat16 stored as uint16 (widened exactly)
 * Lists mode (how many eviction lists a sequence has): 0 = one shared list,
 * 1 = one per layer, 2 = one per (layer, KV head); G = 1, L, L*Hkv.
 *
 * Pins (tests/test_oracle_*.py): every function below is pinned to something
 * other than itself -- brute-force enumeration of ordered keep-tuples, closed
 * forms, textbook special cases, a library Philox generator, dense masked
 * attention, the worked example of the paper's replay-mask figure.
 * No function here is "parity unpinned".
 */
#ifndef NGC_ORACLE_H_
#define NGC_ORACLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Philox4x32 with 10 rounds (Salmon et al., SC'11).  ctr[4], key[2] -> out[4]. */
void ngc_oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out);

/* The fixed single-precision logarithm recipe used for the Gumbel transform
 * (x must be a positive normal float). */
float ngc_oracle_dlog(float x);

/* Random 32-bit word -> uniform in (0,1) -> standard Gumbel variate. */
float ngc_oracle_uniform(uint32_t x);
float ngc_oracle_gumbel(uint32_t x);

/* Perturbed key of unit i of list `list` (Section 4.3: logit + Gumbel noise). */
float ngc_oracle_perturbed_key(float logit, uint64_t seed, uint64_t round,
                               uint32_t list, uint32_t i, int greedy);

/* Section 4.3, Gumbel-top-k.  Per list (b, gi): the n_protect[b] leading units
 * are always kept; budget[b]-n_protect[b] further units are drawn as the
 * largest perturbed keys among units [n_protect[b], n[b]).
 *   logits      [B][G][n_max] fp32
 *   kept_order  [B][G][k_max]  drawn units in descending key order (sigma), -1 padded
 *   kept_sorted [B][G][k_max]  all kept units ascending, -1 padded
 *   keep_mask   [B][G][n_max]  1 = kept (may be NULL)
 *   status      [B][G]         0 ok, 1 bad counts, 2 NaN logit (list skipped; may be NULL)
 * list_base is the global index of list (0,0) (for sharded batches). */
int ngc_oracle_sample_evict(const float* logits, const int32_t* n, const int32_t* n_protect,
                            const int32_t* budget, int B, int G, int n_max, int k_max,
                            uint64_t seed, uint64_t round, uint32_t list_base, int greedy,
                            int32_t* kept_order, int32_t* kept_sorted, uint8_t* keep_mask,
                            int32_t* status);

/* Eq. (1): log-probability of the ordered keep sequence, evaluated literally:
 * one log-sum-exp over the not-yet-selected candidates per step.  O(K*N).
 *   logits [n_batches][B][G][n_max], n/n_protect/budget [n_batches][B],
 *   kept_order [n_batches][B][G][k_max], logp [n_batches][B][G]. */
int ngc_oracle_evict_logprob(const float* logits, const int32_t* n, const int32_t* n_protect,
                             const int32_t* budget, const int32_t* kept_order,
                             int n_batches, int B, int G, int n_max, int k_max, double* logp);

/* Gradient of Eq. (1) with respect to the logits (the eviction half of the policy-gradient loss of
 * Section 4.4 differentiates this log-probability), one softmax over the remaining candidates per
 * step.  grad_logp [n_batches][B][G] (NULL = ones) scales each list; grad_logits
 * [n_batches][B][G][n_max] double out: 0 for protected units and units beyond n[b]. */
int ngc_oracle_evict_logprob_grad(const float* logits, const int32_t* n, const int32_t* n_protect,
                                  const int32_t* budget, const int32_t* kept_order, const double* grad_logp,
                                  int n_batches, int B, int G, int n_max, int k_max, double* grad_logits);

/* Same quantity through the running remaining-mass scan the paper alludes to
 * after Eq. (1) (O(N)); accumulates the remaining mass by addition from the
 * tail.  Cross-checked against the literal form in the tests. */
int ngc_oracle_evict_logprob_scan(const float* logits, const int32_t* n, const int32_t* n_protect,
                                  const int32_t* budget, const int32_t* kept_order,
                                  int n_batches, int B, int G, int n_max, int k_max, double* logp);

/* Section 4.1, physical eviction (what is not kept is gone): out-of-place definition.  For
 * every (layer, head, sequence) strip, row j of k_out/v_out is the j-th kept
 * token in ascending original position.  Units are `block` tokens wide (last
 * unit may be short).  new_lens[b] = number of kept tokens.  k_out/v_out have
 * the same layout as k/v; rows >= new_lens[b] are left untouched.
 * Returns 0, or 3 if a kept list is invalid, 5 if lists of one sequence keep
 * different token counts. */
int ngc_oracle_compact_kv(const void* k, const void* v, const int64_t* seq_off, const int32_t* lens,
                          int L, int B, int Hkv, int d, int dtype,
                          const int32_t* kept_sorted, const int32_t* budget, int k_max,
                          int lists, int block,
                          void* k_out, void* v_out, int32_t* new_lens);

/* Decode attention over the surviving entries.  If new_k/new_v are non-NULL
 * the row is first appended at position lens[b] of each (layer, KV head) strip
 * of layers [layer_begin, layer_end) and is visible to its own query.
 *   q [L][B][Hq][d], new_k/new_v [L][B][Hkv][d] (cache dtype), out [L][B][Hq][d] double.
 * lens[b] is incremented when new rows were given and layer_end == L. */
int ngc_oracle_decode_attn(void* k, void* v, const int64_t* seq_off, int32_t* lens,
                           int L, int B, int Hq, int Hkv, int d, int dtype,
                           const void* q, const void* new_k, const void* new_v,
                           int layer_begin, int layer_end, double scale, double* out);

/* Section 4.2: attention-based eviction scores, block-averaged.
 *   q_recent [L][B][Hq][w][d] (cache dtype); query j of the window sits at
 *   absolute position lens[b]-w+j and sees keys at positions <= its own.
 *   logits   [B][G][n_max] double; units beyond ceil(lens[b]/block) untouched.
 * log_transform: 0 -> s_j, 1 -> log s_j. */
int ngc_oracle_score_evict(const void* k, const int64_t* seq_off, const int32_t* lens,
                           int L, int B, int Hq, int Hkv, int d, int dtype,
                           const void* q_recent, int w, int block, int lists, int log_transform,
                           double* logits, int n_max);

/* Gradient of ngc_oracle_score_evict's logits with respect to q_recent and k (Section 4.4: the
 * eviction loss reaches the model through the scores; Section 4.5 recomputes them on the autograd
 * graph).  grad_logits [B][G][n_max]; grad_q [L][B][Hq][w][d] and grad_k [L][Hkv][R][d] double out
 * (zero where nothing contributes). */
int ngc_oracle_score_evict_grad(const void* k, const int64_t* seq_off, const int32_t* lens,
                                int L, int B, int Hq, int Hkv, int d, int dtype,
                                const void* q_recent, int w, int block, int lists, int log_transform,
                                const double* grad_logits, int n_max, double* grad_q, double* grad_k);

/* Number of OpenMP threads the oracle will use. */
int ngc_oracle_threads(void);

#ifdef __cplusplus
}
#endif
#endif
