/*
 * fkv - budgeted KV-cache eviction and decode attention for one B200 (sm_100a).
 *
 * C ABI of the library built from paper_2602_03203_b200/csrc.  The calls are
 * the paper's statement of the problem (Section 3.1): a cache with budget B
 * that grows by appended (k, v) pairs, is pruned back to B by a learned
 * per-(layer, KV-head) scorer, and is attended over by the decode queries:
 *
 *     fkv_init_cache(shapes, budget)  fkv_append(k, v)  fkv_evict(layer)  fkv_decode_attn(q)
 *
 * Conventions
 *   - Every function returns FKV_OK (0) or a negative fkv_status.  Nothing
 *     throws, nothing is printed.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are host
 *     pointers; a pointer documented "host or dev" may be either.
 *   - All device work is enqueued on the caller's stream (a cudaStream_t passed
 *     as void*); calls return without synchronising unless they say "syncs".
 *     Calls on one cache must be issued on ONE stream, or be ordered by the
 *     caller; two calls on one cache that overlap on the GPU race.
 *   - Host threads: a handle keeps a host-side mirror of the lengths and is not
 *     thread-safe; use one host thread per handle at a time.  The first launch
 *     of each kernel in a process sets its attributes without a lock, so make
 *     the first calls on a device from one thread.
 *   - The library never allocates device memory for a cache.  The caller owns
 *     one device workspace (fkv_workspace_bytes) and keeps it alive until
 *     fkv_destroy; per-call tensors (k, v, q, out, ...) are borrowed until the
 *     enqueued work has run.
 *   - Device-side failures (page pool exhausted, capacity exceeded, a bounded
 *     wait that ran out) do not fault: the kernel skips the work and sets a
 *     bit in a status word that fkv_device_status reads.
 *
 * Terms: one "segment" is the cache of one (sequence, layer, KV head); it
 * holds n "pairs" (slots 0..n-1 in position order).  D = head_dim, g =
 * group_size (query heads per KV head), F = 6g attention features per pair
 * (Appendix B.1), H = scorer_hidden.  bf16 tensors are passed as raw 16-bit
 * patterns.
 */
#ifndef FKV_H
#define FKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FKV_OK = 0,
  FKV_ERR_INVALID_ARG = -1,
  FKV_ERR_WORKSPACE_TOO_SMALL = -2,
  FKV_ERR_CAPACITY = -3,   /* a sequence would exceed max_tokens_per_head */
  FKV_ERR_CUDA = -4,       /* a CUDA call failed; see fkv_last_cuda_error */
  FKV_ERR_NOT_READY = -5,  /* e.g. evict before the scorers are loaded */
  FKV_ERR_DEVICE = -6      /* fkv_device_status found error bits */
} fkv_status;

/* Bits of the device status word (fkv_device_status). */
#define FKV_DEV_POOL_EXHAUSTED 1u /* no free page: the step that needed it was skipped */
#define FKV_DEV_CAPACITY 2u       /* append past max_tokens_per_head was skipped */
#define FKV_DEV_WAIT_TIMEOUT 4u   /* a bounded wait in a kernel ran out */
#define FKV_DEV_BAD_INDEX 8u      /* fkv_compact was given an index outside the segment */

/* Scorer activation sigma.  The paper does not name it (Appendix B.1); ReLU is the default. */
enum { FKV_ACT_RELU = 0, FKV_ACT_SILU = 1, FKV_ACT_GELU_TANH = 2, FKV_ACT_SIGMOID = 3 };

#define FKV_ALL_LAYERS (-1)

typedef struct fkv_cache fkv_cache; /* opaque, host side */

typedef struct {
  int32_t num_layers;
  int32_t num_kv_heads;
  int32_t group_size;          /* g, 1..8 */
  int32_t head_dim;            /* D, 64 or 128 */
  int32_t max_batch;           /* sequences, at most 256 (the efficiency table of Section 4.3 runs up to 96) */
  int32_t page_size;           /* pairs per page; must be 16 */
  int32_t scorer_hidden;       /* H; must be 16 (Section 4.1) */
  int32_t activation;          /* FKV_ACT_* */
  int32_t budget;              /* B for every sequence (fkv_set_budget overrides per sequence) */
  int32_t recent_keep;         /* R: most recent pairs never evicted (the paper's L; 0 = plain top-B) */
  int32_t max_tokens_per_head; /* capacity of one segment, n <= this */
  int32_t num_pages;           /* pages in the pool; 0 = enough for every segment at capacity
                                  plus the transient copies of an all-layer eviction */
  int32_t feature_window;      /* W: decode queries kept on record per (layer, sequence) for the attention
                                  features of Appendix B.1 (a multiple of 8, at most 256;
                                  the paper's update length L, e.g. 256); 0 = the library does not
                                  maintain the features */
} fkv_config;

/* Bytes of device workspace fkv_init_cache needs for this config. */
int fkv_workspace_bytes(const fkv_config *cfg, size_t *bytes);

/*
 * init_cache(shapes, budget) - Section 3.1.  Carves the caller's device
 * workspace (dev, 256-byte aligned, `bytes` long) into the page pool, page
 * tables, lengths, scorer blocks and scratch, and clears it on `stream`.
 * The handle is host memory owned by the library until fkv_destroy.
 */
int fkv_init_cache(const fkv_config *cfg, void *dev_workspace, size_t bytes, void *stream, fkv_cache **out);
int fkv_destroy(fkv_cache *c);

/* Empty every segment and return all pages to the pool (scorers and budgets stay). */
int fkv_reset(fkv_cache *c, void *stream);

/*
 * Scorer of one (layer, KV head) - Appendix B.1:
 *   phi = sigma(x W1 + b1) W2 + b2,  x = Concat(k, v, a).
 * W1: host, [(2D+F)][H] row-major fp32, rows ordered k | v | a; b1, W2: host
 * [H].  The paper states no precision for the weights; they are taken as
 * fp32.  The 2D rows of W1 that multiply k and v are stored as TWO bf16 values
 * per weight, the rounding (to nearest even) of the weight and the rounding of
 * the remainder, and both are multiplied with the bf16 channels on the tensor
 * cores with fp32 accumulation: a weight enters with about 2^-17 relative
 * error instead of bf16's 2^-9.  The F feature rows, b1, W2, b2 stay fp32.
 * Copies to the device on `stream` from a staging buffer the handle owns
 * (syncs).
 */
int fkv_load_scorer(fkv_cache *c, int layer, int kv_head, const float *W1, const float *b1, const float *W2, float b2,
                    void *stream);

/*
 * Per-sequence budget B - Section 3.1 states the problem with one budget B per cache; the batched
 * configurations give every sequence its own (B = half its context), so the budget is a property of
 * the sequence.  Host value; takes effect for later fkv_evict calls.
 */
int fkv_set_budget(fkv_cache *c, int seq, int32_t budget, void *stream);

/*
 * Bulk-load one EMPTY (layer, sequence): n pairs per KV head - the cache as the prefill phase leaves
 * it (Section 3.1 starts from a cache that already holds the prompt; the one-shot compression mode of
 * Section 4.4 evicts right after this call).  The paper has no counterpart for the call itself.
 * k, v: dev [Hkv][n][D] bf16; feat: dev [Hkv][n][F] fp32 or NULL (zeros);
 * pos: dev [n] int32 (strictly increasing token positions) or NULL (0..n-1).
 */
int fkv_prefill(fkv_cache *c, int layer, int seq, const void *k, const void *v, const float *feat, const int32_t *pos,
                int32_t n, void *stream);

/*
 * append(k, v) - Section 3.1: one new pair per sequence and KV head of `layer`.
 * k, v: dev [max_batch][Hkv][D] bf16; pos: dev [max_batch] int32 token
 * positions, or NULL: the position after the last stored one (0 for an empty
 * segment).  The feature row of the new pair is zero.  seq_mask: host bit
 * array of the sequences that take part, (max_batch + 63) / 64 words, bit
 * s % 64 of word s / 64; NULL = all.  It is read before the call returns.
 */
int fkv_append(fkv_cache *c, int layer, const void *k, const void *v, const int32_t *pos, const uint64_t *seq_mask,
               void *stream);

/*
 * Overwrite the attention features a_n (Appendix B.1: six per query head and pair) of one (layer,
 * sequence) with values computed elsewhere: feat dev [Hkv][n][F] fp32, n = current length.  For
 * callers that maintain the features themselves (feature_window = 0) and for checks; the paper has no
 * counterpart for the call itself.
 */
int fkv_set_features(fkv_cache *c, int layer, int seq, const float *feat, void *stream);

/*
 * evict(layer) - Section 3.1 with the deterministic Top-K action: for every
 * segment of `layer` (or of all layers, FKV_ALL_LAYERS) with n > B, score the
 * pairs, keep the R most recent and the B - R best-scoring of the others
 * (higher score first, then lower slot; -0 = +0, NaN lowest), and compact K, V,
 * features and positions of the kept pairs, in position order, into fresh
 * pages.  Afterwards n = B.  Segments with n <= B are left untouched.
 */
int fkv_evict(fkv_cache *c, int layer, void *stream);

/*
 * evict(layer) with the paper's SAMPLED action - Section 3.1, second equation,
 * and Appendix B.2: D = Multinomial_E(Softmax(Top_2E(-Phi))), s' = s \ D.  For
 * every segment with n > B, E = n - B pairs are evicted: the candidates are
 * the 2E competing pairs with the lowest scores (ties: the higher slot ranks
 * lower; all competing pairs if there are fewer than 2E), and E of them are
 * drawn without replacement with probabilities softmax(-score).  The draws use
 * the CALLER'S randomness: noise holds standard Gumbel values g = -log(-log u),
 * u uniform in (0, 1); the candidate of rank j in slot order uses g_j, and the
 * E candidates with the largest (-score + g_j), compared in fp32, are evicted
 * (Gumbel-top-k, which is sampling without replacement from the softmax; ties:
 * the higher slot is evicted).  Everything else is as in fkv_evict.  With all
 * g = 0 this is fkv_evict.
 *
 * noise: dev fp32 [layers of the call][max_batch][Hkv][noise_stride] (one
 * layer, or all layers in order for FKV_ALL_LAYERS); noise_stride must be at
 * least min(2E, n - R) for every segment that is evicted, else
 * FKV_ERR_INVALID_ARG.  The library draws no random numbers itself.
 */
int fkv_evict_sampled(fkv_cache *c, int layer, const float *noise, int32_t noise_stride, void *stream);

/*
 * evict(layer) with a BASELINE score in place of the learned scorer - Appendix E.2.  The score of a
 * pair is one column of its attention features, averaged over the g query heads of the KV head
 * (summed in head order, divided by g, fp32): column FKV_FEATURE_CUM_SUM is H2O (cumulative
 * attention), FKV_FEATURE_WINDOW8 is SnapKV as the paper uses it (attention of the final 8 tokens).
 * Selection, compaction and (with a feature window) the feature refresh are those of fkv_evict; no
 * scorer needs to be loaded.
 */
#define FKV_FEATURE_WINDOW8 0
#define FKV_FEATURE_WINDOW16 1
#define FKV_FEATURE_WINDOW32 2
#define FKV_FEATURE_WINDOW_CHUNK 3
#define FKV_FEATURE_CUM_SUM 4
#define FKV_FEATURE_CUM_DECAY 5
int fkv_evict_by_feature(fkv_cache *c, int layer, int32_t column, void *stream);

/*
 * evict(layer) with the R-KV baseline score - Appendix E.2: "R-KV also takes into account the redundancy among
 * tokens": the window attention score and a token-to-token similarity are weighed 0.1 and 0.9.  The paper gives
 * the weights and no formula; this library's reading:
 *     score_i = lambda_attn * a_i - lambda_sim * s_i
 *     a_i = the SnapKV score above (feature FKV_FEATURE_WINDOW8 averaged over the g query heads),
 *     s_i = the largest cosine between the stored key k_i and the key of ANOTHER pair of the same segment
 *           (0 if either key is the zero vector, or the segment has one pair),
 * so a pair with a near-duplicate elsewhere in the cache is evicted before an equally attended unique one.
 * No normalisation of either term.  Cost: the n x n products of a segment's keys, 2 n^2 D flops, on the tensor
 * cores.  Features must be finite.  Everything else is as in fkv_evict_by_feature.  FKV_RKV_LAMBDA_* are the
 * paper's weights.  fkv_score_rkv is the score alone (layout as fkv_score).
 * Errors beyond those of fkv_evict_by_feature: FKV_ERR_CUDA if the driver's tensor-map encoder cannot be reached or
 * refuses the page pool's geometry, or if the device cannot place clusters of two thread blocks (the contraction
 * runs on pairs of SMs); fkv_last_cuda_error has the text.  No pair is evicted or moved in that case.
 */
#define FKV_RKV_LAMBDA_ATTN 0.1f
#define FKV_RKV_LAMBDA_SIM 0.9f
int fkv_evict_rkv(fkv_cache *c, int layer, float lambda_attn, float lambda_sim, void *stream);
int fkv_score_rkv(fkv_cache *c, int layer, float lambda_attn, float lambda_sim, float *scores_out, void *stream);

/*
 * decode_attn(q) - Appendix A: out[s][h] = sum_i softmax_i(scale <q[s][h], k_i>) v_i
 * over all retained pairs i of the KV head that query head h belongs to
 * (h / g).  q, out: dev [max_batch][Hkv*g][D] bf16.  scale 0 means 1/sqrt(D).
 * Sequences with n = 0 get zeros.
 */
int fkv_decode_attn(fkv_cache *c, int layer, const void *q, void *out, float scale, void *stream);

/*
 * append(k, v) followed by decode_attn(q) on `layer`, as ONE kernel launch
 * (Section 3.1 + Appendix A): the new pair of every participating sequence is
 * stored at slot n and attended together with the n retained pairs.  Arguments
 * as in fkv_append and fkv_decode_attn; the result equals the two calls made
 * one after the other.
 */
int fkv_append_decode_attn(fkv_cache *c, int layer, const void *k, const void *v, const int32_t *pos,
                           const uint64_t *seq_mask, const void *q, void *out, float scale, void *stream);

/*
 * One decode token through every layer, in layer order: for l = 0 .. L-1,
 * fkv_append_decode_attn(k[l], v[l], q[l]) -> out[l].  k, v: dev
 * [L][max_batch][Hkv][D] bf16; q, out: dev [L][max_batch][Hkv*g][D] bf16; pos:
 * dev [max_batch] or NULL (as fkv_append).  One launch per layer, issued from
 * native code.  Every layer's k, v and q must be complete when the call is
 * enqueued: the layers do not depend on one another here, so the launches of
 * layers 1 .. L-1 are allowed to run alongside the launch before them
 * (programmatic dependent launch), and out[l] is complete only when the whole
 * step is (the next work on the stream is ordered after all of it).  For
 * engines that have all layers' tensors at hand, and for benchmarks of the
 * attention side alone.
 *
 * Stream capture: fkv_append_decode_attn and fkv_decode_step only enqueue
 * kernels, so they may be recorded into a CUDA graph.  Every replay appends one
 * more pair per sequence from the recorded k / v / q buffers: the kernel reads
 * the lengths on the device, divides a segment's pages over the recorded number
 * of splits whatever its length has become, and skips an append past
 * max_tokens_per_head (FKV_DEV_CAPACITY).  The host's copy of the lengths does
 * not see replays: call fkv_sync_lengths after the last replay and before any
 * other call of this library.
 */
int fkv_decode_step(fkv_cache *c, const void *k, const void *v, const int32_t *pos, const void *q, void *out,
                    float scale, void *stream);

/* ---- staged entry points: one kernel each, for per-step checks ---- */

/*
 * The scorer alone - Appendix B.1: phi_n = sigma(Concat(k_n, v_n, a_n) W1 + b1) W2 + b2 for every pair
 * of `layer`, with the (layer, KV head)'s own weights (Section 3.1: one scoring model per layer and
 * attention group).  scores_out dev [max_batch][Hkv][cap] fp32, cap = fkv_score_stride.
 */
int fkv_score(fkv_cache *c, int layer, float *scores_out, void *stream);
/*
 * The selection alone - Section 3.1: the most recent R pairs stay, the others are pruned back to
 * B - R by score (the lowest scores are evicted; the Top-K row of the paper's sampling ablation, i.e.
 * the deterministic action; ties: higher score, then lower slot).  From given scores (dev, layout as
 * fkv_score writes them) writes for each segment the kept slots, ascending, to idx_out dev
 * [max_batch][Hkv][cap] int32 and their number min(B, n) to kept_count_out dev [max_batch][Hkv].
 */
int fkv_select(fkv_cache *c, int layer, const float *scores_in, int32_t *idx_out, int32_t *kept_count_out,
               void *stream);
/* Selection by the sampled action of fkv_evict_sampled from given scores; noise dev [max_batch][Hkv][noise_stride]. */
int fkv_select_sampled(fkv_cache *c, int layer, const float *scores_in, const float *noise, int32_t noise_stride,
                       int32_t *idx_out, int32_t *kept_count_out, void *stream);
/*
 * The compaction alone - Section 3.1's state update s' = s \ D: the kept pairs' K, V, feature and
 * position rows move, in order, into fresh pages and the segment's length becomes the kept count.
 * By given ascending slot lists (dev, layout as fkv_select writes them; every sequence must have the
 * same count on all its heads).  Syncs (reads the new lengths back).
 */
int fkv_compact(fkv_cache *c, int layer, const int32_t *idx, const int32_t *kept_count, void *stream);

/*
 * Attention features a_n of Appendix B.1, maintained by the library when feature_window > 0.
 * Every fkv_append_decode_attn / fkv_decode_step records the token's queries, their softmax
 * statistics and the number of pairs they saw (the last W tokens since the last eviction).
 * fkv_evict / fkv_evict_sampled then refresh the features of the segments they evict, before
 * scoring: per query head, in this order inside a_n,
 *   windows 8, 16, 32: (1/w) sum over the last w recorded queries of the softmax probability
 *                      the head gave the pair (0 for queries older than the pair),
 *   window = chunk:    the same mean over all recorded queries of the chunk (the chunk's score),
 *   direct sum:        previous value + chunk score,
 *   decayed sum:       0.9 * previous value + chunk score,
 * and start a new chunk.  With no query on record (e.g. right after fkv_prefill) the stored
 * features are used as they are.  The paper gives one sentence on these features; mean versus sum,
 * and what a chunk is, are this library's reading of it.
 * fkv_update_features does the refresh alone for `layer` (all its sequences), without closing the
 * chunk - a staged entry point for checks.  FKV_ERR_NOT_READY if feature_window is 0.
 */
int fkv_update_features(fkv_cache *c, int layer, void *stream);

/* Row stride, in elements, of the score and index arrays above. */
int fkv_score_stride(const fkv_cache *c, int32_t *cap);

/*
 * Dense copy of one segment: k, v dev [n][D] bf16, feat dev [n][F], pos dev [n]; any may be NULL.
 * The paper has no counterpart: a read-out for checks and for moving a cache elsewhere.
 */
int fkv_export_head(fkv_cache *c, int layer, int seq, int kv_head, void *k, void *v, float *feat, int32_t *pos,
                    void *stream);

/* Current lengths of `layer`: host_out [max_batch] (host mirror, no device access). */
int fkv_get_lengths(const fkv_cache *c, int layer, int32_t *host_out);

/*
 * Reads the device status word and free-page count (syncs `stream`); clears the word.
 * When it returns FKV_ERR_DEVICE, a kernel has skipped work the host had already counted (an append, or
 * a whole eviction step), so the host's copy of the lengths may be ahead of the device: call
 * fkv_sync_lengths (or fkv_reset) before any other call on this handle.
 */
int fkv_device_status(fkv_cache *c, uint32_t *status_bits, int32_t *free_pages, void *stream);

/*
 * Re-read the lengths of every layer from the device into the host mirror
 * (syncs).  For callers that restored a saved copy of the workspace.
 */
int fkv_sync_lengths(fkv_cache *c, void *stream);

/*
 * Per-kernel timing of fkv_evict.  While on, fkv_evict records CUDA events on
 * the caller's stream around its kernels; fkv_get_evict_timing waits for the
 * last recorded set and returns milliseconds for
 * {plan, score, select (both passes of the sampled action), compact, commit, feature refresh}.
 */
int fkv_set_timing(fkv_cache *c, int on);
int fkv_get_evict_timing(fkv_cache *c, float ms_out[6]);

/* Number of kernel launches this handle has enqueued so far. */
int fkv_launch_count(const fkv_cache *c, uint64_t *launches);

/*
 * Decode attention without any allocation (the paper has no counterpart; this
 * is a service entry point of the library).
 *
 * For callers that may not allocate device memory: code running inside a
 * memory pool that was sized once and frozen, a serving process that accounts
 * for every byte of HBM itself, a plug-in that is handed tensors and nothing
 * else.  Such a caller cannot provide the workspace fkv_init_cache needs, so
 * this call takes dense tensors and keeps its split-K partials in a fixed
 * array inside the library image (about 1.1 MB of HBM on every GPU that loads
 * the library, held until the process exits).  It calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 *   out[h] = sum_i softmax_i(scale <q[h], k[h / g][i]>) v[h / g][i],  i < n
 *
 * q, out: dev [num_kv_heads * group_size][head_dim] bf16; k, v: dev
 * [num_kv_heads][n][head_dim] bf16, dense row-major; scale 0 means
 * 1/sqrt(head_dim).  Same arithmetic as fkv_decode_attn (fp32 online softmax,
 * bf16 result), for one sequence.
 *
 * k and v must be 8-byte aligned (FKV_ERR_INVALID_ARG otherwise).  This is a
 * service path: it reads one row per warp and step and is far slower than
 * fkv_decode_attn for long sequences.
 *
 * Limits: head_dim 64 or 128 (else FKV_ERR_INVALID_ARG); 1 <= n <=
 * FKV_NOALLOC_MAX_PAIRS, num_kv_heads <= FKV_NOALLOC_MAX_KV_HEADS, group_size
 * <= 8 - beyond them the call does nothing and returns FKV_ERR_CAPACITY.
 *
 * The first call on a device looks up the array's device address (once per
 * device, with that device current); make that first call before any stream
 * capture begins.  All calls share the one array, which keeps the previous
 * call's partials (the call clears the only part that must start at zero):
 * two calls that overlap on the GPU - different streams, or different
 * threads without ordering - race on it.  Order them on one stream.
 */
#define FKV_NOALLOC_MAX_PAIRS (1 << 20)
#define FKV_NOALLOC_MAX_KV_HEADS 16
int fkv_decode_attn_dense_noalloc(const void *q, const void *k, const void *v, int32_t n, int32_t num_kv_heads,
                                  int32_t group_size, int32_t head_dim, float scale, void *out, void *stream);

/*
 * Golden Eviction labels - Section 3.2, Eq. 3-5: the supervision targets of the scorer, from the full
 * attention matrix of ONE attention group (no cache handle involved).
 *   attn: dev fp32 [g][T][T] attention probabilities of the group's g heads, row = query position,
 *         column = key position.
 * Query rows are cut into blocks of L starting at the first eviction position B + L (the last block
 * zero-padded): M = ceil((T - B) / L) - 1 blocks = eviction steps (fkv_golden_steps).  Block score =
 * average over the g heads and the block's L rows; future score alpha[t][i] = maximum of the block
 * scores of pair i over blocks t .. M; retained set of step t = the B - L pairs with the largest
 * alpha[t][.] among the B cached ones (those retained at step t - 1 plus the L tokens that just left
 * the recent window; [0, B) at step 1; ties: lower position).  The L newest tokens are kept by the
 * protocol and are not listed.
 *   alpha_out: dev fp32 [M][T] (row t - 1 = step t); kept_out: dev int32 [M][B - L], ascending.
 * B <= 8192 (FKV_ERR_CAPACITY beyond); M = 0 does nothing.  fkv_golden_select is the last step alone,
 * from given future scores.
 */
int fkv_golden_steps(int32_t T, int32_t B, int32_t L);
int fkv_golden_eviction(const float *attn, int32_t g, int32_t T, int32_t B, int32_t L, float *alpha_out,
                        int32_t *kept_out, void *stream);
int fkv_golden_select(const float *alpha, int32_t T, int32_t B, int32_t L, int32_t M, int32_t *kept_out, void *stream);

/* Text of the last CUDA error seen by this library on this thread ("" if none). */
const char *fkv_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FKV_H */
