/*
 * spark.h -- C ABI of the SparK hot path on one NVIDIA B200 (sm_100a).
 *
 * SparK prunes the key cache per token along the channel axis and restores the
 * pruned entries while the decode query is scored.  Two calls carry the method:
 *
 *   spark_compress      observation-window queries + full K/V  ->  packed cache
 *   spark_decode_attn   decode query + packed cache            ->  attention output
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller unless marked
 *     "host".  The library allocates nothing and keeps no state between calls.
 *   - Work is enqueued on the caller's stream (`spark_stream_t` is a
 *     `cudaStream_t`); nothing synchronises except spark_read_status.
 *   - Errors the host can see (null pointers, shapes, sizes) are returned as a
 *     spark_status BEFORE any launch.  Errors only the device can see (a page
 *     id outside the pool, a bounded wait that ran out) are recorded in the
 *     status word at the start of the workspace and the kernel returns without
 *     touching the bad address; read them with spark_read_status.
 *   - head_dim must be 128, page_tokens 16, 1 <= n_q_heads / n_kv_heads <= 8.
 *   - Alignment: q, k_new, v_new, qnorm, out and the page pool must be 16-byte aligned (the kernels use
 *     16-byte vector accesses), workspaces 256-byte aligned; a misaligned pointer is refused with
 *     SPARK_ERR_BAD_SHAPE.  max_blocks must not exceed INT32_MAX / 16.
 *
 * Packed cache.  The cache is a pool of fixed-size pages.  One page holds
 * `page_tokens` consecutive tokens of ONE KV head of one sequence:
 *     kept key values (ascending channel order) | 128-bit channel mask per token
 *     | mu_pruned per token (fp32) | dense value rows
 * or, with value-channel pruning (keep_v < head_dim), kept value entries and a second
 * 128-bit mask per token in place of the dense value rows.
 * `block_table[b][h][i]` is the pool index of the page with tokens
 * [16 i, 16 i + 16) of sequence b, KV head h.  Every call that takes a block table also accepts NULL for a
 * CONTIGUOUS cache: unit (b, h) then owns the max_blocks consecutive pages starting at
 * (b * n_kv_heads + h) * max_blocks, n_pool_pages must cover them all, and the decode step saves the table
 * lookups.  The byte layout inside a page is
 * private to the library (spark_page_bytes gives its size; spark_unpack_pages
 * turns pages back into logical arrays).  Slots of a page past the end of the
 * sequence are zero.
 */
#ifndef SPARK_H_
#define SPARK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *spark_stream_t;            /* a cudaStream_t; NULL is the legacy default stream */

typedef enum {
    SPARK_OK = 0,
    SPARK_ERR_NULL = 1,                  /* a required pointer is NULL                        */
    SPARK_ERR_BAD_SHAPE = 2,             /* inconsistent or out-of-range sizes                */
    SPARK_ERR_UNSUPPORTED = 3,           /* head_dim != 128, page_tokens != 16, dtype, G > 8  */
    SPARK_ERR_WORKSPACE = 4,             /* workspace missing, misaligned or too small        */
    SPARK_ERR_CUDA = 5,                  /* a CUDA runtime call failed (launch, attribute)    */
    SPARK_ERR_DEVICE_BOUNDS = 6,         /* device saw a page id / length out of range        */
    SPARK_ERR_DEVICE_TIMEOUT = 7         /* a bounded device-side wait ran out                */
} spark_status;

typedef enum { SPARK_F32 = 0, SPARK_BF16 = 1 } spark_dtype;

typedef struct {
    int32_t batch;          /* B, sequences                                                   */
    int32_t n_q_heads;      /* Hq                                                             */
    int32_t n_kv_heads;     /* Hkv; query head i reads KV head i / (Hq / Hkv)                 */
    int32_t head_dim;       /* D = 128                                                        */
    int32_t window;         /* W, observation-window queries per query head                   */
    int32_t keep;           /* T, kept key channels per token, 1..D                           */
    int32_t page_tokens;    /* 16                                                             */
    int32_t dtype;          /* spark_dtype of q, k, v and of the packed values                */
    int32_t token_budget;   /* 0: no eviction; else tokens kept per KV head, window included  */
    int32_t pool_kernel;    /* odd max-pool width of the eviction votes (7); budget > 0 only  */
    float   qnorm_eps;      /* floor of |mean window query|; 0 selects 1e-12                  */
    float   softmax_scale;  /* 0 selects 1/sqrt(head_dim)                                     */
    int64_t n_pool_pages;   /* pages in the pool; every block-table entry must be below it    */
    int32_t flags;          /* bit set of spark_flags (0: none)                               */
    int32_t keep_v;         /* T_v, kept value channels per token; 0 or D: values stay dense   */
    int32_t select;         /* spark_select: how the kept key channels of a token are chosen  */
    float   top_p;          /* SPARK_SELECT_TOP_P: share of a token's total saliency to keep   */
    int32_t n_groups;       /* SPARK_SELECT_GROUPS: rank groups, 1..8                         */
    float   group_prune[8]; /* SPARK_SELECT_GROUPS: pruning ratio per group, most salient first */
    int32_t recovery;       /* spark_recovery: distribution that restores the pruned entries   */
    uint32_t seed;          /* sampled recovery: seed of the per-entry draws                   */
} spark_params;

/* spark_params.select -- the ratio-free variants of Sec. "Ablation Studies" ("Adaptive Variants").
 * In every mode `keep` is the capacity of a token's slot list in the page: the number of kept channels
 * under SPARK_SELECT_FIXED, an upper bound under the two others.
 *   SPARK_SELECT_TOP_P   (SparK-p) per token, rank the channels by saliency and keep the fewest, at least
 *                        one and at most `keep`, whose saliencies add up to top_p times the token's total
 *                        (sums in double, most salient first).
 *   SPARK_SELECT_GROUPS  (SparK-g) per token, cut the saliency ranks into n_groups segments of D / n_groups
 *                        ranks (the first D % n_groups segments get one more); segment i keeps its
 *                        floor((1 - group_prune[i]) * size_i) most salient channels.  `keep` must be at
 *                        least their sum (spark_group_keep).  The paper lists the ratios and the group
 *                        counts but not how the groups are formed; ranks per token is this library's reading. */
typedef enum { SPARK_SELECT_FIXED = 0, SPARK_SELECT_TOP_P = 1, SPARK_SELECT_GROUPS = 2 } spark_select;

/* spark_params.recovery -- the recovery distributions of Sec. "Channel Recovery".  The sampled ones use the
 * all-channel mean and population deviation of a token's saliencies (App. "Caching Pruned Channel
 * Statistics"), which the page then carries per token (8 more bytes).  One draw per pruned entry, a pure
 * function of (seed, sequence, KV head, token, channel): the recovered keys are fixed for the life of the
 * cache.  Sampled recovery needs dense value rows (keep_v == 0).
 *   SPARK_RECOVER_DEGENERATE   w~ = mu_pruned (the default everywhere in the paper)
 *   SPARK_RECOVER_GAUSSIAN     w~ ~ N(mu, sigma^2), not clamped
 *   SPARK_RECOVER_EXPONENTIAL  w~ ~ Exp(1 / mu), i.e. mean mu */
typedef enum { SPARK_RECOVER_DEGENERATE = 0, SPARK_RECOVER_GAUSSIAN = 1, SPARK_RECOVER_EXPONENTIAL = 2 } spark_recovery;

/* spark_params.flags */
typedef enum {
    /* spark_decode_attn only.  Launch the step so that it may begin while the kernel enqueued before it
     * on the same stream is still draining (programmatic dependent launch): the page stream -- pages,
     * block table, packed_lens -- is read at once, while q, qnorm, out, lse and the workspace are touched
     * only after that preceding kernel has completed.  Set it only when the preceding kernel does not
     * write the packed cache, the block table or packed_lens (a projection that produces q is fine).
     * Results are identical with and without the flag. */
    SPARK_FLAG_OVERLAP_PREVIOUS = 1,
    /* spark_decode_attn_host only.  q_host, out_host (and lse_host) are page-locked host memory that the device
     * can address (cudaHostAlloc / cudaHostRegister under unified addressing): the kernel writes the result
     * across the bus itself, no staging copies are enqueued, and q_dev / out_dev / lse_dev may be NULL.  The
     * query takes one of two routes.  bf16 storage, degenerate recovery, dense value rows and a query of at
     * most 24 KB (B * Hq * 256 bytes): its bytes are read DURING THE CALL and travel to the GPU inside the
     * kernel launch, so q_host must hold the query when the call is made (not merely when the stream gets
     * there) and may be reused as soon as the call returns.  Otherwise the kernel reads q_host across the bus
     * during the step (stream order, as without the flag).  If the runtime cannot give a device address for
     * a buffer it needs, the call returns SPARK_ERR_BAD_SHAPE before anything is enqueued. */
    SPARK_FLAG_HOST_MAPPED = 2
} spark_flags;

/* T = floor((1 - ratio) * head_dim): the paper's kept-channel count (Sec. "Problem
 * Formulation", below Eq. (cal)).  Host only.  Returns -1 for ratio outside [0, 1). */
int32_t spark_keep_count(int32_t head_dim, double ratio);

/* Kept channels per token under SPARK_SELECT_GROUPS: sum over the groups of floor((1 - prune[i]) * size_i).
 * Host only.  -1 on bad arguments. */
int32_t spark_group_keep(int32_t head_dim, int32_t n_groups, const float *group_prune);

/* Bytes of one page for these parameters (uses head_dim, keep, page_tokens, dtype).
 * Host only.  0 on unsupported parameters. */
size_t spark_page_bytes(const spark_params *p);

/* Bytes of the whole page pool: n_pool_pages * spark_page_bytes(p), plus -- under SPARK_SELECT_TOP_P -- an
 * int32 per pool page behind the pages (256-byte aligned) in which the library keeps how many slot rows of
 * the page are in use; the decode step then copies only that much of each page.  The caller allocates the
 * pool with this size.  Host only.  0 on unsupported parameters. */
size_t spark_pool_bytes(const spark_params *p);

/* Bytes the method itself has to read per token and KV head in one decode step:
 * kept key values + mask + mu_pruned + the dense value row, or with value-channel pruning the
 * kept value entries + their mask (the roofline numerator).  Host only. */
size_t spark_algorithmic_bytes_per_token(const spark_params *p);

/* Workspace sizes.  `max_seq_tokens` bounds seq_lens (before eviction).  Either
 * output pointer may be NULL.  Host only. */
spark_status spark_workspace_bytes(const spark_params *p, int64_t max_seq_tokens,
                                   size_t *compress_bytes, size_t *decode_bytes);

/* Zero a workspace.  Must be enqueued once before the first call that uses the
 * workspace; the calls leave it ready for the next one. */
spark_status spark_workspace_init(void *workspace, size_t workspace_bytes, spark_stream_t stream);

/*
 * spark_compress -- prefill-side pruning (Sec. "SparK": "Saliency Measurement and
 * Unstructured Pruning"; statistics of App. "Caching Pruned Channel Statistics").
 *
 * For every sequence b and KV head h:
 *   q-bar[j] = mean of the G*W window queries of the G query heads that share h
 *   a[j]     = max(|q-bar[j]|, qnorm_eps)                       -> qnorm[b][h][j]
 *   w[t][j]  = a[j] * |K[t][j]|      one round-to-nearest fp32 multiply
 *   kept_t   = the `keep` channels of largest w[t][.], lower channel first on ties
 *   mu[t]    = mean of w[t][j] over the pruned channels (0 when keep == head_dim)
 * and the page of token t receives K[t][kept_t] (bit-identical, ascending channel
 * order), the mask, mu[t] and V[t][:].
 *
 * With 0 < keep_v < head_dim the value rows are pruned as well (App. "Pruning Value Cache
 * Channels"): per token the keep_v value channels of largest |V[t][j]| are kept (lower channel
 * first on ties), bit-identical, in ascending channel order, with their own 128-bit mask; the
 * other entries are dropped and count as zero in the weighted sum of spark_decode_attn.
 *
 * With token_budget > 0 the tokens are first reduced per KV head to
 * min(S_b, token_budget) by observation-window attention votes (softmax of the
 * window queries against all earlier keys, causal inside the window, summed over
 * the group and the window, max-pooled with pool_kernel, top-(budget - W) of the
 * prefix plus the W window tokens, original order); the paper cites this step
 * from its base eviction method (App. "Implementation") and does not define it.
 *
 *   q_win        [B][Hq][W][D] contiguous; the window is the LAST W tokens of each sequence
 *   k, v         element (b,h,t,j) at b*stride_b + h*stride_h + t*stride_t + j (in elements)
 *   seq_lens     [B] int32, tokens per sequence (<= max_seq_tokens)
 *   pages        OUT page pool, n_pool_pages * spark_page_bytes(p) bytes, 16-byte aligned
 *   block_table  [B][Hkv][max_blocks] int32 pool indices; entries are read for
 *                i < ceil(packed_len_b / 16)
 *   qnorm        OUT [B][Hkv][D] fp32
 *   packed_lens  OUT [B] int32, tokens per KV head after eviction (= seq_lens when budget == 0)
 *   kept_tokens  OUT optional [B][Hkv][token_budget] int32 original positions (budget > 0), else NULL
 *   workspace    scratch of at least compress_bytes (spark_workspace_bytes), 256-byte aligned
 */
spark_status spark_compress(const spark_params *p,
                            const void *q_win, const void *k, const void *v,
                            int64_t stride_b, int64_t stride_h, int64_t stride_t,
                            const int32_t *seq_lens, int32_t max_seq_tokens,
                            void *pages, const int32_t *block_table, int32_t max_blocks,
                            float *qnorm, int32_t *packed_lens, int32_t *kept_tokens,
                            void *workspace, size_t workspace_bytes, spark_stream_t stream);

/*
 * spark_append -- decode-time append of one token per sequence (Sec. "Preliminaries": the new key and
 * value are concatenated to the cache, K <- Cat[K, k]).  The paper prunes during prefill and does not say
 * how keys appended later are treated; here the new key is pruned at once with the sequence's prefill
 * statistics: w[j] = qnorm[j] * |k[j]|, the `keep` largest channels are kept, mu is the mean of the rest --
 * exactly what spark_compress would have stored for that token given the same window queries.  With
 * value-channel pruning (keep_v) the new value row is pruned by |v[j]| in the same way.
 *
 *   k_new, v_new   [B][Hkv][D] contiguous, dtype as the cache, 16-byte aligned
 *   pages, block_table, max_blocks, qnorm   as used by spark_compress / spark_decode_attn; the page that
 *                  holds token index packed_lens[b] must be listed in the block table (a fresh page is
 *                  cleared by this call)
 *   packed_lens    IN/OUT [B]: every sequence with room (packed_lens[b] < 16 * max_blocks) grows by one;
 *                  a full sequence is left unchanged and SPARK_ERR_DEVICE_BOUNDS is recorded
 *   workspace      at least 256 bytes, 256-byte aligned (status word only)
 */
spark_status spark_append(const spark_params *p, const void *k_new, const void *v_new,
                          void *pages, const int32_t *block_table, int32_t max_blocks,
                          const float *qnorm, int32_t *packed_lens,
                          void *workspace, size_t workspace_bytes, spark_stream_t stream);

/*
 * spark_append_block -- the same for n_new tokens per sequence at once: k_new, v_new are [B][Hkv][n_new][D]
 * and every sequence grows by n_new tokens (by as many as fit; SPARK_ERR_DEVICE_BOUNDS is recorded when some do
 * not).  This is how keys that a caller has kept DENSE for a while -- the paper's K <- Cat[K, k] of Sec.
 * "Preliminaries" taken literally -- enter the pruned cache block by block.  0 <= n_new <= 65535.
 */
spark_status spark_append_block(const spark_params *p, const void *k_new, const void *v_new, int32_t n_new,
                                void *pages, const int32_t *block_table, int32_t max_blocks,
                                const float *qnorm, int32_t *packed_lens,
                                void *workspace, size_t workspace_bytes, spark_stream_t stream);

/*
 * spark_merge_attn -- attention over the union of two disjoint token sets from the two partial results
 * (Sec. "Preliminaries": softmax attention; the log-sum-exp identity that also merges the token splits inside
 * spark_decode_attn).  With w_x = exp(lse_x - lse), lse = log(exp(lse_a) + exp(lse_b)):
 *     out = w_a * out_a + w_b * out_b
 * A side with lse = -inf (no tokens) contributes nothing; both empty gives out = 0, lse = -inf.  Typical use:
 * a sequence held as a pruned prefix (one cache) plus a dense tail of recently appended tokens (a second cache
 * with keep = head_dim): decode both with their lse and merge.
 *   out_a, out_b, out  [batch][n_q_heads][head_dim] fp32, 16-byte aligned (out may alias an input)
 *   lse_a, lse_b       [batch][n_q_heads] fp32;  lse  OUT optional
 */
spark_status spark_merge_attn(int32_t batch, int32_t n_q_heads, int32_t head_dim,
                              const float *out_a, const float *lse_a, const float *out_b, const float *lse_b,
                              float *out, float *lse, spark_stream_t stream);

/*
 * spark_decode_attn -- one decode step over the packed cache (Sec. "Channel Recovery"
 * with the degenerate distribution, then the attention of Sec. "Preliminaries").
 *
 * For every sequence b and query head i (KV head h = i / G):
 *   K~[t][j] = K[t][j] if channel j of token t was kept, else mu[t] / a[j]
 *   s[t]     = softmax_scale * sum_j q[i][j] * K~[t][j]
 *   out[i]   = sum_t softmax_t(s)[t] * V[t][:]          over t < packed_lens[b]
 *              (with value-channel pruning, V[t][c] counts as 0 where channel c of token t was dropped)
 * Accumulation is fp32; the softmax is computed online over token splits that are
 * merged by their log-sum-exp.  A sequence of length 0 yields out = 0, lse = -inf.
 *
 *   q            [B][Hq][D] contiguous, dtype as the cache
 *   pages, block_table, max_blocks, packed_lens, qnorm   as written by spark_compress
 *   out          OUT [B][Hq][D] fp32
 *   lse          OUT optional [B][Hq] fp32, natural-log sum-exp of the scaled scores
 *   workspace    at least decode_bytes, 256-byte aligned, initialised once by spark_workspace_init
 */
spark_status spark_decode_attn(const spark_params *p, const void *q,
                               const void *pages, const int32_t *block_table, int32_t max_blocks,
                               const int32_t *packed_lens, const float *qnorm,
                               float *out, float *lse,
                               void *workspace, size_t workspace_bytes, spark_stream_t stream);

/*
 * spark_decode_attn_host -- the same decode step for a caller whose query and result live in HOST memory
 * (Sec. "Channel Recovery" / "Preliminaries" as above; only the transport differs).  Enqueues, in this order
 * on `stream`: the copy of q_host to q_dev, spark_decode_attn on q_dev, the copy of out_dev to out_host (and
 * of lse_dev to lse_host when both are given).  Nothing is synchronised: the results are in out_host once
 * the stream has reached this point.
 *
 *   (With SPARK_FLAG_HOST_MAPPED the two copies are replaced by direct device access to the host buffers.)
 *   q_host             HOST [B][Hq][D], dtype as the cache; page-locked memory lets the copy run asynchronously
 *   q_dev              DEVICE staging for the query, same size, 16-byte aligned
 *   out_dev            DEVICE [B][Hq][D] fp32, 16-byte aligned;  out_host  HOST, same size
 *   lse_dev, lse_host  optional, both NULL or both given, [B][Hq] fp32
 *   every other argument as for spark_decode_attn; errors are returned before anything is enqueued
 *   except a failing copy (SPARK_ERR_CUDA).
 */
spark_status spark_decode_attn_host(const spark_params *p, const void *q_host, void *q_dev,
                                    const void *pages, const int32_t *block_table, int32_t max_blocks,
                                    const int32_t *packed_lens, const float *qnorm,
                                    float *out_dev, float *out_host, float *lse_dev, float *lse_host,
                                    void *workspace, size_t workspace_bytes, spark_stream_t stream);

/*
 * spark_decode_attn_noalloc -- spark_decode_attn for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the call above, same arithmetic.)
 *
 * Who needs it: code that is handed device tensors but no allocator -- a serving loop whose memory
 * was divided up once at start-up, a plug-in inside another runtime, a framework section in which
 * cudaMalloc is forbidden.  Such a caller can supply inputs and outputs but not the scratch that split
 * decoding needs, so this variant uses a fixed scratch array that lives in the library's own device
 * image (about 1.3 MB per GPU that loads the library, held until the process exits).  It calls no
 * cudaMalloc, cudaFree or allocating library routine.
 *
 *   - Limit: batch * n_kv_heads <= 64 (any group size up to 8).  Larger problems are refused with
 *     SPARK_ERR_WORKSPACE before anything is enqueued; use spark_decode_attn with your own workspace.
 *   - The first call on each device looks up the array's device address (the device must be current).
 *     Make that first call outside any stream capture.
 *   - Every call shares the one array.  The entry point clears the status word and the tickets on the
 *     stream before launching; two calls that overlap on the GPU (different streams, no dependency)
 *     would race on it and are not supported.  Device-side errors are not readable through
 *     spark_read_status for this variant (there is no caller-visible workspace).
 *   - All other arguments, results and error codes are those of spark_decode_attn.
 */
spark_status spark_decode_attn_noalloc(const spark_params *p, const void *q,
                                       const void *pages, const int32_t *block_table, int32_t max_blocks,
                                       const int32_t *packed_lens, const float *qnorm,
                                       float *out, float *lse, spark_stream_t stream);

/*
 * spark_unpack_pages -- pages back to logical arrays (what the paper calls the pruned
 * key matrix K^, the mask S and mu_pruned; Sec. "Saliency Measurement and Unstructured
 * Pruning").  For inspection and tests; any output may be NULL.
 *
 *   mask   OUT [B][Hkv][max_tokens][4] uint32, bit (j % 32) of word (j / 32) <=> channel j kept
 *   mu     OUT [B][Hkv][max_tokens] fp32
 *   vals   OUT [B][Hkv][max_tokens][keep] in the cache dtype, ascending channel order
 *   v      OUT [B][Hkv][max_tokens][D] in the cache dtype (dropped value entries read back as 0)
 * Rows t >= packed_lens[b] are written as zeros.
 */
spark_status spark_unpack_pages(const spark_params *p, const void *pages,
                                const int32_t *block_table, int32_t max_blocks,
                                const int32_t *packed_lens, int32_t max_tokens,
                                uint32_t *mask, float *mu, void *vals, void *v,
                                spark_stream_t stream);

/* spark_unpack_stats -- the all-channel saliency statistics a page carries under a sampled recovery
 * distribution (App. "Caching Pruned Channel Statistics": mean mu_i and population deviation sigma_i).
 *   mu_all, sigma_all  OUT [B][Hkv][max_tokens] fp32, zeros for rows t >= packed_lens[b]; either may be NULL.
 * SPARK_ERR_UNSUPPORTED when recovery is SPARK_RECOVER_DEGENERATE (the page has no such section). */
spark_status spark_unpack_stats(const spark_params *p, const void *pages,
                                const int32_t *block_table, int32_t max_blocks,
                                const int32_t *packed_lens, int32_t max_tokens,
                                float *mu_all, float *sigma_all, spark_stream_t stream);

/* spark_unpack_value_masks -- the per-token value-channel masks (App. "Pruning Value Cache Channels").
 *   vmask  OUT [B][Hkv][max_tokens][4] uint32, bit (j % 32) of word (j / 32) <=> value channel j kept;
 *          all ones for live tokens when the values are dense, zeros for rows t >= packed_lens[b]. */
spark_status spark_unpack_value_masks(const spark_params *p, const void *pages,
                                      const int32_t *block_table, int32_t max_blocks,
                                      const int32_t *packed_lens, int32_t max_tokens,
                                      uint32_t *vmask, spark_stream_t stream);

/* Synchronise `stream` and return the status word of a workspace (SPARK_OK when no
 * kernel recorded an error).  Debug and tests only. */
spark_status spark_read_status(const void *workspace, spark_stream_t stream);

/* Number of kernels the last successful spark_decode_attn / spark_compress call of this
 * thread enqueued (host only; for launch accounting in benchmarks). */
int32_t spark_last_launch_count(void);

/* Library version: major * 10000 + minor * 100 + patch.  Host only. */
int32_t spark_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPARK_H_ */
