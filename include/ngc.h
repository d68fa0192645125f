/*
 * ngc.h -- C ABI of the B200 (sm_100a) hot path of Neural Garbage Collection:
 * batched rollout decoding over a KV cache that the policy itself prunes.
 *
 * One eviction round is   ngc_score_evict -> ngc_sample_evict -> ngc_evict_logprob
 * -> ngc_compact_kv,   after which generation continues with
 * ngc_decode_attn_ragged over the surviving entries (paper Section 4.1: the
 * cache grows during generation and is pruned at each round).
 *
 * Conventions
 * -----------
 * - Plain C.  Host-side state: the last CUDA error code (per thread) and one
 *   flag per device recording that a kernel family has been configured there
 *   (the first call of a kernel family on each device sets its shared-memory
 *   limit, which CUDA stores per device; make that first call outside any
 *   stream capture).  Device-side state: none, except the built-in scratch
 *   array of ngc_decode_attn_ragged_static (see there).
 * - Every data pointer is a DEVICE pointer owned by the caller unless the
 *   comment says "host".  The library never allocates, frees or synchronises;
 *   scratch comes from a caller-supplied workspace sized by
 *   ngc_workspace_bytes() (ngc_decode_attn_ragged_static alone uses its own
 *   array instead).  Every call only enqueues work on `stream` (a
 *   cudaStream_t, which must belong to the current device) and returns.
 * - Return value: NGC_OK or a negative ngc_status.  Invalid host-visible
 *   arguments are refused before anything is launched.  Problems only visible
 *   on the device (a budget larger than the list, a NaN logit, a corrupt kept
 *   list, a full strip) are written to *dev_status (int32 in device memory,
 *   first error wins, 0 = none; may be NULL) and the offending list / strip /
 *   sequence is skipped.  Kernels never trap and every wait inside them is
 *   bounded.
 * - "Lists": a sequence has G eviction lists; G = 1 (one decision shared by all
 *   layers and heads), L (one per layer, the paper's setting: Section 4.1 has
 *   every layer evict an equal share of its entries but choose them on its
 *   own), or L*Hkv (one per layer and KV head).  List gi of sequence b is
 *   row b*G + gi of every [B][G][...] array.
 * - "Units": eviction acts on units of `block` consecutive tokens (Section 4.2,
 *   block-level evictions); the last unit of a sequence may be short.
 *
 * Cache layout
 * ------------
 *   k, v    : [L][Hkv][R][d] elements; R rows per (layer, KV head) plane.
 *   seq_off : int64 [B+1]; sequence b owns rows seq_off[b] .. seq_off[b+1] of
 *             every plane (its capacity); seq_off[0] = 0, seq_off[B] = R.
 *   lens    : int32 [B]; the first lens[b] rows of a strip are alive.  With
 *             lens_lists != 0 the cache holds one length per (sequence, list) instead:
 *             int32 [B][G] for that ngc_lists mode, and the strips of list gi of
 *             sequence b have lens[b*G + gi] alive rows.  The paper evicts per layer
 *             in units of several tokens, and a short last unit that one layer keeps
 *             and another evicts leaves the layers with different lengths.
 * A (layer, head, sequence) strip is therefore T x d contiguous rows, which
 * decode streams linearly and compaction moves row by row.  Rows at or beyond
 * lens[b] hold unspecified bytes.
 */
#ifndef NGC_H_
#define NGC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* ngc_stream;   /* == cudaStream_t */

typedef enum {
  NGC_OK = 0,
  NGC_ERR_INVALID_ARG = -1,   /* null pointer, negative size, inconsistent shape */
  NGC_ERR_UNSUPPORTED = -2,   /* shape / dtype combination not built */
  NGC_ERR_WORKSPACE = -3,     /* workspace missing or smaller than ngc_workspace_bytes() */
  NGC_ERR_CUDA = -4,          /* a CUDA call failed; code in ngc_last_cuda_error() */
  NGC_ERR_STATIC_SCRATCH = -5 /* launch needs more scratch than the built-in static array holds */
} ngc_status;

/* values written to *dev_status */
typedef enum {
  NGC_DEV_OK = 0,
  NGC_DEV_BAD_COUNTS = 1,     /* not 0 <= n_protect <= budget <= n <= n_max, or budget > k_max */
  NGC_DEV_NAN_LOGIT = 2,      /* a candidate logit is NaN */
  NGC_DEV_BAD_KEPT = 3,       /* kept list out of range, repeated or not ascending */
  NGC_DEV_STRIP_FULL = 4,     /* append would exceed the sequence's row capacity */
  NGC_DEV_LISTS_DISAGREE = 5, /* lists of one sequence keep different token counts */
  NGC_DEV_TIMEOUT = 6,        /* a bounded wait inside a kernel ran out */
  NGC_DEV_DEBUG_BOUNDS = 7    /* bounds-checking build only: a kernel computed an index outside its array */
} ngc_dev_status;

typedef enum { NGC_F32 = 0, NGC_BF16 = 1 } ngc_dtype;
typedef enum { NGC_LISTS_SHARED = 0, NGC_LISTS_PER_LAYER = 1, NGC_LISTS_PER_LAYER_KVHEAD = 2 } ngc_lists;
typedef enum { NGC_OP_SCORE = 0, NGC_OP_SAMPLE = 1, NGC_OP_LOGPROB = 2, NGC_OP_COMPACT = 3, NGC_OP_DECODE = 4,
               NGC_OP_SCORE_BACKWARD = 5 } ngc_op;

/* Describes the cache; owns nothing.  `rows` and `max_len` are host copies the
 * launch geometry needs: rows = seq_off[B]; max_len >= every length at the
 * time of the call (a loose bound such as the largest capacity is fine; it
 * only sizes grids and workspaces). */
typedef struct {
  void* k;
  void* v;
  const int64_t* seq_off;
  int32_t* lens;
  int64_t rows;
  int32_t L, B, Hq, Hkv, d;   /* Hq % Hkv == 0; d in {64, 128} */
  int32_t dtype;              /* ngc_dtype of k, v, queries and new rows */
  int32_t max_len;
  int32_t lens_lists;         /* 0: lens[B]; NGC_LISTS_PER_LAYER / _KVHEAD: lens[B][G] of that mode.  Calls that
                                 take an eviction `lists` mode need lens_lists == 0 or == lists. */
} ngc_cache;

/* Library version (major*10000 + minor*100 + patch). */
int ngc_version(void);
/* Text for an ngc_status (host string, never NULL). */
const char* ngc_strerror(int status);
/* cudaError_t of the most recent NGC_ERR_CUDA on this host thread (0 = none). */
int ngc_last_cuda_error(void);

/* Bytes of workspace `op` needs for this cache / list shape (0 = none).  For
 * NGC_OP_SAMPLE and NGC_OP_LOGPROB only c->B (sequences, times rounds for the
 * log-prob) is read from the cache descriptor; pass G, n_max, k_max as in the
 * call.  The workspace must be 256-byte aligned; its contents need not be
 * preserved between calls, and calls sharing a workspace must be stream-ordered. */
size_t ngc_workspace_bytes(int op, const ngc_cache* c, int G, int n_max, int k_max);

/* Number of token-range splits ngc_decode_attn_ragged uses for a call over
 * `layers` layers of this cache (1 = every strip is handled by one CTA and no
 * combine kernel runs).  Host-only planning query. */
int ngc_decode_splits(const ngc_cache* c, int layers);

/*
 * Eviction scores -- Section 4.2 ("Parameterizing eviction actions" and
 * "Coarsening the action space").  For every list: psi_t = mean, over the
 * query heads feeding the list and the w most recent queries, of the softmax
 * attention weight (scale 1/sqrt(d)) that query puts on alive key t; then
 * s_j = mean of psi over the tokens of unit j.
 *   q_recent [L][B][Hq][w][d], cache dtype.  Window query j sits at absolute
 *            position lens[b]-w+j and sees keys at positions <= its own; when
 *            lens[b] < w only the last lens[b] queries are used.
 *   lists    which heads are averaged: SHARED = all layers and heads,
 *            PER_LAYER = the Hq heads of the layer (the paper), PER_LAYER_KVHEAD
 *            = the Hq/Hkv heads of one KV group.
 *   logits   [B][G][n_max] fp32 out.  With one length per sequence, units >=
 *            ceil(lens[b]/block) are untouched.  With a length per list
 *            (lens_lists == lists) the sequence is scored on the units of its
 *            LONGEST list, n_b = max over its lists of ceil(len/block): a shorter
 *            list gets -inf in the units it lacks (never drawn by
 *            ngc_sample_evict, no mass in Eq. (1)); units >= n_b are untouched.
 *   n_units_out  int32 [B] out, may be NULL: n_b, the unit count per sequence to
 *            pass to ngc_sample_evict / ngc_evict_logprob as `n` (for one length
 *            per sequence simply ceil(lens[b]/block)).
 *   log_transform  0: logit = s_j (the paper's literal reading); 1: logit = log s_j.
 * Requires n_max >= ceil(max_len/block).  Reads K only.
 */
int ngc_score_evict(const ngc_cache* c, const void* q_recent, int w, int block, int lists,
                    int log_transform, float* logits, int n_max, int32_t* n_units_out,
                    void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/* Number of kernels one ngc_score_evict call enqueues for this cache and window (host-only planning query, for
 * launch counting). */
int ngc_score_evict_launches(const ngc_cache* c, int w);

/*
 * Gradient of the eviction scores with respect to the recent queries and the
 * keys -- Sections 4.4 and 4.5: the eviction loss reaches the model through
 * the scores, which the replay pass recomputes with gradients enabled.  The chain
 * rule through the block mean, the average over attention rows and the
 * softmax of ngc_score_evict:
 *   grad_logits   [B][G][n_max] fp32 upstream gradient (e.g. from ngc_evict_logprob_backward)
 *   logits        the forward output; read only when log_transform != 0 (else may be NULL)
 *   grad_q_recent [L][B][Hq][w][d] fp32 out (zero for window queries before the sequence start)
 *   grad_k        [L][Hkv][R][d] out, cache dtype; rows >= lens[b] are not written
 * Other arguments as in ngc_score_evict.  Built for bf16 caches with d = 128 and at most 40
 * (head, query) rows per KV head (Hq/Hkv * w <= 40); NGC_ERR_UNSUPPORTED otherwise.  K is read
 * twice and grad_k written once.  Workspace: ngc_workspace_bytes(NGC_OP_SCORE_BACKWARD, ...).
 */
int ngc_score_evict_backward(const ngc_cache* c, const void* q_recent, int w, int block, int lists, int log_transform,
                             const float* logits, const float* grad_logits, int n_max,
                             float* grad_q_recent, void* grad_k,
                             void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/*
 * Sampling the keep set -- Section 4.3 (Gumbel-top-k): perturbed key =
 * logit + Gumbel noise; keep the budget largest.  The n_protect[b] leading
 * units are always kept and take no part in the draw; budget[b] counts them.
 * Noise: Philox4x32-10 with key = seed and counter = (i >> 2, list_base + b*G
 * + gi, round low, round high); unit i takes output word i & 3; the word
 * becomes an odd multiple of 2^-24 in (0,1) and then a Gumbel variate through a
 * fixed sequence of correctly rounded fp32 operations, so that the draw does
 * not depend on launch geometry, on the batch sharding or on the machine.
 * Ties (equal fp32 keys): smaller index first.  greedy != 0 drops the noise
 * (Section 5.1, evaluation uses deterministic top-k).
 *   logits      [B][G][n_max] fp32
 *   n, n_protect (may be NULL = 0), budget : int32 [B]
 *   kept_order  [B][G][k_max] out: the budget-n_protect drawn units, largest key
 *               first (the sequence sigma of Eq. (1)); -1 padded
 *   kept_sorted [B][G][k_max] out: all kept units ascending; -1 padded
 *   keep_mask   [B][G][n_max] out, 1 = kept (may be NULL)
 * A list with bad counts or a NaN candidate logit is reported in *dev_status
 * and gets all -1 / 0 outputs.
 */
int ngc_sample_evict(const float* logits, const int32_t* n, const int32_t* n_protect,
                     const int32_t* budget, int B, int G, int n_max, int k_max,
                     uint64_t seed, uint64_t round, uint32_t list_base, int greedy,
                     int32_t* kept_order, int32_t* kept_sorted, uint8_t* keep_mask,
                     void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/*
 * Log-probability of the drawn sequence -- Eq. (1) of Section 4.3:
 *   log p(sigma | s) = sum_j [ s_sigma_j - log sum_{t not in sigma_1..sigma_{j-1}} exp s_t ],
 * over the non-protected units of each list, evaluated with the running
 * remaining-mass scan the paper mentions right after the equation, in fp64.
 * Rounds can be flattened into the leading dimension (the policy-gradient
 * recompute of Section 4.4 evaluates all rounds of a rollout at once).
 *   logits [n_batches][B][G][n_max] fp32; n, n_protect (NULL = 0), budget
 *   int32 [n_batches][B]; kept_order [n_batches][B][G][k_max];
 *   logp [n_batches][B][G] fp64 out (NaN for a list reported in *dev_status).
 */
int ngc_evict_logprob(const float* logits, const int32_t* n, const int32_t* n_protect,
                      const int32_t* budget, const int32_t* kept_order,
                      int n_batches, int B, int G, int n_max, int k_max, double* logp,
                      void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/*
 * Gradient of that log-probability with respect to the logits -- what the
 * eviction half of the policy-gradient loss (Section 4.4, L_mem: the sum over
 * layers and rounds of -log pi(sigma) * advantage) sends back into the scores:
 *   d log p / d s_i = [i in sigma] - exp(s_i) * sum_{j : i not drawn before step j} 1 / rem_j ,
 * rem_j = the mass still present at step j (the same scan as the forward call).
 *   grad_logp   fp64 [n_batches][B][G] upstream gradient per list, or NULL (= 1)
 *   grad_logits fp32 [n_batches][B][G][n_max] out; every entry of a list is
 *               written: 0 for protected units and units >= n[b], NaN for a
 *               list reported in *dev_status.
 * Other arguments as in ngc_evict_logprob.  Lists with more than about 24 K
 * drawn units are refused with NGC_ERR_UNSUPPORTED.
 */
int ngc_evict_logprob_backward(const float* logits, const int32_t* n, const int32_t* n_protect,
                               const int32_t* budget, const int32_t* kept_order, const double* grad_logp,
                               int n_batches, int B, int G, int n_max, int k_max, float* grad_logits,
                               void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/*
 * Replay visibility -- Appendix A.3 ("Reconstructing Replay Attention Masks
 * from Retention Decisions") and the replay-mask figure of Section 4.5.  The
 * training pass must show every token exactly the keys it saw at rollout time:
 * a query generated after round r sees kept_r (what round r left alive) plus,
 * causally, the tokens generated since.  This call turns the stored decisions
 * of all R rounds -- kept units in the coordinates of the cache at that round
 * -- into kept_r as ORIGINAL token positions, one ascending list per (round,
 * list), instead of the paper's dense B x T x T masks.
 *   kept_sorted  [R][B][G][k_max] as written by ngc_sample_evict at round r
 *   budget       [R][B] kept units;  alive_before [R][B] tokens alive when round
 *                r fired (lens[b] at that time), or [R][B][G] with per_list != 0 (caches
 *                with a length per list);  total_before [R][B] sequence
 *                length when round r fired (the tokens appended since the last
 *                round are the positions just below it)
 *   block        tokens per unit;  alive_max (host) >= every alive_before
 *   alive_pos    [R][B][G][k_max*block] out, ascending, -1 padded
 *   alive_count  [R][B][G] out (tokens), -1 for a list that failed
 * A list with inconsistent counts or a corrupt kept list is reported in
 * *dev_status and gets -1 from the failing round on.
 */
int ngc_replay_visibility(const int32_t* kept_sorted, const int32_t* budget, const int32_t* alive_before,
                          const int32_t* total_before, int R, int B, int G, int k_max, int block, int alive_max,
                          int per_list, int32_t* alive_pos, int32_t* alive_count, int32_t* dev_status, ngc_stream stream);

/*
 * Replay attention -- Section 4.5: one pass over ALL tokens of a rollout in
 * which every query sees exactly the keys it saw when it was generated, so
 * that token and eviction log-probabilities are recomputed on-policy.  The
 * masks of Appendix A.3 are not materialised: the query at position t attends
 * to kept_r (alive_pos of the last round that fired at or before t, from
 * ngc_replay_visibility) and, causally, to the tokens from that round's
 * boundary up to t itself; queries before the first round are plain causal.
 *   c            the FULL sequences: k, v [L][Hkv][R][d] hold every token in original
 *                order, lens[b] = T_b tokens (bf16, d = 128)
 *   q            [L][B][Hq][t_max][d] bf16; rows >= lens[b] are ignored
 *   alive_pos    [n_rounds][B][G][kt_max], alive_count [n_rounds][B][G], total_before
 *                [n_rounds][B] (ascending per sequence); n_rounds = 0: causal attention
 *   lists        how G maps to (layer, KV head), as everywhere
 *   out          [L][B][Hq][t_max][d] fp32 or bf16; rows >= lens[b] are not written
 * fp32 scores, softmax and accumulation; probabilities rounded to bf16 for P*V.
 * Needs no workspace.  Runs on the tcgen05 tensor cores with accumulators in
 * tensor memory; every wait inside is bounded (NGC_DEV_TIMEOUT).
 */
int ngc_replay_attn(const ngc_cache* c, const void* q, int t_max,
                    const int32_t* alive_pos, const int32_t* alive_count, const int32_t* total_before,
                    int n_rounds, int kt_max, int lists, float scale, void* out, int out_dtype,
                    int32_t* dev_status, ngc_stream stream);

/* ngc_replay_attn with the device path chosen by the caller (same arguments, same contract; for
 * measuring one path against the other).  AUTO is what ngc_replay_attn runs: the tcgen05 kernel
 * (S and O accumulators in tensor memory, one CTA per 128 query tokens of two heads).  MMA_SYNC is
 * the earlier warp-level kernel (64 query tokens of one head per CTA). */
typedef enum { NGC_REPLAY_ATTN_AUTO = 0, NGC_REPLAY_ATTN_MMA_SYNC = 1, NGC_REPLAY_ATTN_TCGEN05 = 2 } ngc_replay_attn_path;
int ngc_replay_attn_variant(const ngc_cache* c, const void* q, int t_max,
                            const int32_t* alive_pos, const int32_t* alive_count, const int32_t* total_before,
                            int n_rounds, int kt_max, int lists, float scale, void* out, int out_dtype, int variant,
                            int32_t* dev_status, ngc_stream stream);

/*
 * Physical eviction -- Section 4.1 (entries that are not kept are gone for good).  In place:
 * in every (layer, KV head, sequence) strip of K and V the tokens of the kept
 * units move to the front in ascending original order, and lens[b] becomes
 * the number of kept tokens.  Bit-exact row moves; rows beyond the new length
 * are unspecified afterwards.
 *   kept_sorted [B][G][k_max] ascending unit indices (as written by
 *   ngc_sample_evict); budget int32 [B]; lists says how G maps to (layer, head).
 * Errors leave whole sequences alone: with one length per sequence (lens_lists
 * == 0), a sequence that has a corrupt list (NGC_DEV_BAD_KEPT), or whose lists
 * would keep different token counts (NGC_DEV_LISTS_DISAGREE: units of several
 * tokens with a short last unit that some lists keep and others evict), is
 * reported and none of its strips moves; its lens[b] and every row are as
 * before the call.  With a length per list (lens_lists == lists) the lists are
 * independent: a corrupt list leaves its own strips and length untouched.
 * (While the call runs, lens[b] of such a sequence briefly holds a negative
 * marker; it is restored before the call's last kernel ends.)
 */
int ngc_compact_kv(ngc_cache* c, const int32_t* kept_sorted, const int32_t* budget, int k_max,
                   int lists, int block, int32_t* dev_status, ngc_stream stream);

/*
 * Decode attention over the surviving entries -- Section 4.1 (after a round,
 * generation goes on with only what was kept).  For layers
 * [layer_begin, layer_end): if new_k/new_v are given, the new token's K/V row
 * is first written at position lens[b] of each strip and is visible to its
 * own query; then out = softmax(scale * q K^T) V over the alive rows, one
 * pass, split along tokens.  lens[b] is incremented (once) by the call whose
 * layer_end == L when new rows were given.
 *   q      [L][B][Hq][d] cache dtype; new_k, new_v [L][B][Hkv][d] cache dtype or both NULL
 *   out    [L][B][Hq][d] of out_dtype (NGC_F32, or NGC_BF16 for a bf16 cache);
 *          only the layers of the range are written; an empty strip gives zeros.
 * bf16 caches: fp32 scores, softmax and accumulation; the probabilities are
 * rounded to bf16 for the P*V product.
 */
int ngc_decode_attn_ragged(ngc_cache* c, const void* q, const void* new_k, const void* new_v,
                           int layer_begin, int layer_end, float scale,
                           void* out, int out_dtype,
                           void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/*
 * Paged variant -- Section 4.2 remarks that evicting whole blocks fits paged
 * KV caches: with one eviction unit = one page, evicting is
 * an edit of a page table and no K/V row moves.
 *
 *   k, v       : [L][Hkv][B * pages_cap][page][d] elements (bf16, d = 128)
 *   page_table : int32 [B][G][pages_cap]; the j-th page of tokens of list gi of
 *                sequence b lives in physical page  b * pages_cap + page_table[b][gi][j]
 *                of every (layer, KV head) plane the list covers.  Each row of the
 *                table is a permutation of 0 .. pages_cap-1: entries at and beyond
 *                ceil(lens[b] / page) name the sequence's free pages.
 *   lens       : int32 [B] alive tokens (same for every list of b), or int32 [B][G] with
 *                lens_per_list != 0 (a partly filled last page that one list keeps and
 *                another evicts leaves them with different lengths)
 *   lists      : ngc_lists, fixes G and which planes a list covers
 *   page       : tokens per page, 32 or 64
 */
typedef struct {
  void* k;
  void* v;
  int32_t* page_table;
  int32_t* lens;
  int32_t L, B, Hq, Hkv, d;
  int32_t dtype;
  int32_t page, pages_cap, lists;
  int32_t lens_per_list;
} ngc_paged_cache;

/*
 * ngc_score_evict over a paged cache: units are pages (block = page), the
 * lists are the cache's own (c->lists); K is read page by page through the
 * table.  logits [B][G][n_max], n_max >= pages_cap; n_units_out as in
 * ngc_score_evict (may be NULL).  Workspace as for
 * NGC_OP_SCORE of a contiguous cache with rows = B * pages_cap * page and
 * max_len = pages_cap * page.
 */
int ngc_score_evict_paged(const ngc_paged_cache* c, const void* q_recent, int w, int log_transform,
                          float* logits, int n_max, int32_t* n_units_out, void* ws, size_t ws_bytes,
                          int32_t* dev_status, ngc_stream stream);

/*
 * Eviction on a paged cache: for every list the pages named by kept_sorted
 * (ascending unit = page indices, as written by ngc_sample_evict) move to the
 * front of the list's page-table row in that order, the other pages follow as
 * free pages, and lens[b] becomes the number of kept tokens (a partly filled
 * last page stays last if it is kept).  No K/V row is touched.  A corrupt list
 * leaves its row and lens[b] unchanged and is reported in *dev_status.
 */
int ngc_evict_pages(ngc_paged_cache* c, const int32_t* kept_sorted, const int32_t* budget, int k_max,
                    int32_t* dev_status, ngc_stream stream);

/*
 * ngc_decode_attn_ragged over a paged cache: same arguments, results and
 * append semantics; the token tiles are fetched page by page through the
 * table.  The appended row goes to position lens[b] of the list's pages (a
 * sequence is full at pages_cap * page tokens).  Workspace as for
 * NGC_OP_DECODE of a cache with the same L, B, Hq, Hkv.
 */
int ngc_decode_attn_paged(ngc_paged_cache* c, const void* q, const void* new_k, const void* new_v,
                          int layer_begin, int layer_end, float scale,
                          void* out, int out_dtype,
                          void* ws, size_t ws_bytes, int32_t* dev_status, ngc_stream stream);

/*
 * ngc_decode_attn_ragged without a caller-supplied workspace.  (The paper has
 * no counterpart: this entry exists for the library's users, not the method.)
 *
 * Some callers cannot hand the library device scratch memory: code embedded
 * in a host application that has already given every byte of device memory
 * to its own pool, plug-ins that are not allowed to call the CUDA allocator,
 * and latency-critical serving loops where a cudaMalloc (which synchronises
 * the whole device) must never happen.  For them the split partials of the
 * decode kernel live in a scratch array built into the library image
 * (NGC_STATIC_SCRATCH_BYTES of device memory, resident on every GPU that
 * loads the library until the process exits).  The call allocates nothing,
 * frees nothing and calls no allocating routine.
 *
 * Same arguments and results as ngc_decode_attn_ragged, minus ws/ws_bytes.
 * - A launch whose scratch need exceeds NGC_STATIC_SCRATCH_BYTES is refused
 *   with NGC_ERR_STATIC_SCRATCH before anything is enqueued (use the
 *   workspace variant, or narrow the layer range).
 * - The first call on each device looks up the device address of the array
 *   (a one-off host-side set-up on the current device, serialised by a
 *   mutex); make that first call before starting any stream capture.
 * - The array used is the CURRENT device's; a `stream` that belongs to another
 *   device is refused with NGC_ERR_INVALID_ARG.
 * - All calls on a device share the one array, which keeps whatever the last
 *   call left in it.  Nothing in it needs to start at zero (every slot is
 *   written before it is read within a call), but two calls that overlap on
 *   the GPU (different streams without an ordering between them) race on it:
 *   keep calls to this entry stream-ordered.
 */
#define NGC_STATIC_SCRATCH_BYTES (8u << 20)
int ngc_decode_attn_ragged_static(ngc_cache* c, const void* q, const void* new_k, const void* new_v,
                                  int layer_begin, int layer_end, float scale,
                                  void* out, int out_dtype, int32_t* dev_status, ngc_stream stream);

/*
 * Self-test of the bounded wait.  (The paper has no counterpart: this is a
 * diagnostic of the library's own safety contract.)  The streaming kernels wait
 * for their TMA data on mbarriers with a time limit; when a wait runs out the
 * kernel records NGC_DEV_TIMEOUT in *dev_status and runs on to its end.  This
 * call launches one warp that waits, for at most limit_us microseconds
 * (1 .. 100000), on a barrier that nothing ever completes, so that the path
 * can be exercised on a healthy device: afterwards *dev_status is
 * NGC_DEV_TIMEOUT (if it was 0 before), *waited_ns (device uint64, may be
 * NULL) holds the time spent waiting, and the stream and context are usable as
 * before.  dev_status must not be NULL.
 */
int ngc_selftest_bounded_wait(uint32_t limit_us, int32_t* dev_status, uint64_t* waited_ns, ngc_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* NGC_H_ */
