/*
 * liblocks -- per-step decode hot path of the LOCKS page-local spectral-summary selector,
 * hand-written CUDA for NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes only.
 *
 * Notation (the paper's): B tokens per page, d head dimension, Hq query heads, Hkv KV heads,
 * G = Hq/Hkv, T tokens of a sequence including the one being decoded, P = ceil(T/B) pages,
 * b token budget per KV head, k = ceil(b/B) page budget, r summary rank.
 *
 * Conventions shared by every call
 *  - Pointers are DEVICE pointers unless the parameter name ends in _host.  The caller owns every
 *    buffer, including the workspace handed to locks_create(); the library allocates no device
 *    memory, never frees caller memory and keeps no caller pointer between calls except the
 *    workspace.
 *  - Every call only enqueues kernels (and, for the *_host variants, async copies) on `stream`
 *    (a cudaStream_t passed as void*), does not synchronise unless stated, and launches a fixed
 *    grid that depends only on the configuration and `batch`: lengths and page tables are read
 *    on the device, so a captured CUDA graph can be replayed as the sequences grow.
 *  - Return value: LOCKS_OK or a negative LOCKS_ERR_* code.  Argument errors are found on the
 *    host before anything is launched.  Problems only the device can see (a block id outside the
 *    cache, a bounded wait that expired) set a sticky status word in the workspace, the affected
 *    kernel skips that piece of work, and locks_poll_status() reports it.  Nothing traps.
 *  - Precondition of locks_select / locks_decode_step: every candidate page (1 .. P-2) of every
 *    request has a summary built by locks_build_summaries (locks_decode_step maintains this).
 */
#ifndef LOCKS_H_
#define LOCKS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LOCKS_OK 0
#define LOCKS_ERR_INVALID_ARG (-1)
#define LOCKS_ERR_UNSUPPORTED (-2)
#define LOCKS_ERR_WORKSPACE (-3)
#define LOCKS_ERR_CUDA (-4)
#define LOCKS_ERR_TIMEOUT (-5)
#define LOCKS_ERR_BAD_BLOCK (-6)
#define LOCKS_ERR_TOO_LARGE (-7)

#define LOCKS_F32 0
#define LOCKS_BF16 1

#define LOCKS_FMT_F32 0 /* summary stored as fp32 mu, V, C                               */
#define LOCKS_FMT_I4 1  /* int4 basis, int8 coefficients + centroid, fp16 scales (r8i4)  */
#define LOCKS_FMT_I8 2  /* int8 basis, int8 coefficients + centroid: the "int8 basis" arm of the paper's rank x
                           precision ablation (App. B); plain fp32-arithmetic kernels                    */
#define LOCKS_FMT_BF16 3 /* bf16 basis, int8 coefficients + centroid: the paper's "r8fp" control (Sec. 4
                           robustness paragraph, App. B); plain fp32-arithmetic kernels                  */

/* How the G query heads of a KV head are combined into one ranking key per page (Sec. 4; ablated in the
 * paper's App. D "GQA combine" table).  The selection (sink + most recent + top k-2 by key, ties to the lower
 * page) is the same for all; page_logshare receives the key.
 *   LOCKS_COMBINE_SHARE_AVG   log mean_g exp(s^_j(q_g) - log Z_g): the paper's rule (Cor. 4)
 *   LOCKS_COMBINE_GROUP_MAX   max_g s^_j(q_g): the largest raw page log-mass of the group
 *   LOCKS_COMBINE_GROUP_MASS  log sum_g exp s^_j(q_g): the group's summed, un-normalised page mass
 *   LOCKS_COMBINE_PER_HEAD    no combine: every query head ranks by its own share and keeps its own k pages (the
 *                             per-head arm of that table: up to G times the attention traffic).  page_ids is then
 *                             [batch][Hq][k], page_count [batch][Hq], page_logshare [batch][Hq][max_pages_per_seq] in
 *                             locks_select and locks_sparse_attend; locks_decode_step and the diagnostics that take a
 *                             page table per KV head return UNSUPPORTED. */
#define LOCKS_COMBINE_SHARE_AVG 0
#define LOCKS_COMBINE_GROUP_MAX 1
#define LOCKS_COMBINE_GROUP_MASS 2
#define LOCKS_COMBINE_PER_HEAD 3

typedef struct locks_ctx locks_ctx;
typedef void *locks_stream; /* cudaStream_t */

typedef struct {
  int32_t head_dim;          /* d; 128                                                        */
  int32_t page_size;         /* B; 16, or 32 | 64 (App. D "Page size": plain fp32 kernels)       */
  int32_t num_q_heads;       /* Hq                                                            */
  int32_t num_kv_heads;      /* Hkv, Hq % Hkv == 0, G = Hq/Hkv <= 16                          */
  int32_t rank;              /* r: I4 format 2|4|8, other formats 1..16                       */
  int32_t summary_fmt;       /* LOCKS_FMT_*                                                   */
  int32_t kv_dtype;          /* LOCKS_F32 | LOCKS_BF16 (K, V, k_new, v_new)                   */
  int32_t q_dtype;           /* LOCKS_F32 | LOCKS_BF16 (q and out); must equal kv_dtype       */
  int32_t max_batch;         /* largest `batch` any call will pass                            */
  int32_t max_pages_per_seq; /* row length of block_table                                     */
  int32_t budget_tokens;     /* b; k = ceil(b/B) >= 2                                         */
  float sm_scale;            /* logit scale, 1/sqrt(d) in the paper                           */
  int32_t combine;           /* LOCKS_COMBINE_*: how a group's heads share one page table (0 = the paper's)   */
} locks_config;

/* Paged KV cache view.  Element (block, kv head, token-in-page, dim) of K lives at
 * k[block*stride_block + head*stride_head + token*stride_token + dim] (strides in ELEMENTS; dims
 * are contiguous), likewise V.  Both [block][head][token][dim] and [block][token][head][dim] fit.
 * For 16-byte vector loads the strides must be multiples of 8 elements and the bases 16-byte
 * aligned. */
typedef struct {
  void *k, *v;
  int64_t stride_block, stride_head, stride_token;
  int32_t num_blocks;
  const int32_t *block_table; /* [max_batch][max_pages_per_seq] logical page -> physical block */
  int32_t *seq_lens;          /* [max_batch] tokens in each sequence (see each call)           */
} locks_kv;

/* Bytes of one stored summary, per (physical block, KV head), padded to a multiple of 16.
 * I4 format: 82 r + 162 payload bytes at B=16, d=128 (978 / 1298 at r = 8, B = 32 / 64;
 * 818 / 490 / 326 at r = 8 / 4 / 2: the
 * paper's stored-payload table, App. C.1), i.e. d r/2 int4 basis + B r int8 coefficients + d int8
 * centroid + (r + B + 1) fp16 scales (Sec. 4 "Build").  F32 format: 4 (d + r d + B r).  I8 format: d r + B r + d +
 * 2 (r + B + 1).  BF16 format: 2 d r + B r + d + 2 (B + 1).  The last two are plain row-major:
 * [basis r x d][coefficients B x r][centroid d][coefficient scales B][basis scales r (I8 only)][centroid scale],
 * integer codes stored offset-binary (byte = code + 128).
 * The summaries buffer is [num_blocks][Hkv][locks_summary_bytes]. 0 on an invalid config. */
size_t locks_summary_bytes(const locks_config *cfg);

/* Bytes of device workspace locks_create() needs for this configuration (256-byte aligned
 * base).  0 on an invalid config. */
size_t locks_workspace_bytes(const locks_config *cfg);

/* Validate the configuration, record it and the workspace pointer, zero the status word (one
 * small async memset on the default stream followed by a synchronise).  The context is a small
 * host object; *out must be released with locks_destroy().  Errors: INVALID_ARG (bad field, NULL),
 * UNSUPPORTED (shape the kernels do not cover: d != 128, B not in {16, 32, 64}, G > 16, mixed dtypes, I4 rank not
 * in {2,4,8}), WORKSPACE (ws_bytes too small or misaligned).  Pages of 32 and 64 tokens run build, select, attend
 * and the decode step on plain fp32 kernels (no tensor-core path); the diagnostics, the KV fake quantiser, the
 * page-sharded calls, the multi-layer build and the allocation-free attention entry point return UNSUPPORTED for
 * them. */
int locks_create(const locks_config *cfg, void *workspace, size_t ws_bytes, locks_ctx **out);
int locks_destroy(locks_ctx *ctx);

/* Summary build (Sec. 4 "Build (once, when a page completes)"): for each request b < batch, each
 * KV head and each COMPLETE page p with page_begin[b] <= p < page_end[b] (p < floor(T_b/B)):
 * centre the page's B keys, eigendecompose the B x B Gram of the deviations, keep r modes
 * (C = U_r Sigma_r, V = D^T U_r Sigma_r^-1, zero modes dropped), quantise and store the blob at
 * summaries[block][head].  page_begin == page_end == NULL: all complete pages.
 * seq_lens[b] = T_b.  Arithmetic fp32. */
int locks_build_summaries(locks_ctx *ctx, const locks_kv *kv, int batch, const int32_t *page_begin,
                          const int32_t *page_end, void *summaries, locks_stream stream);

/* The same build for several layers of a model in ONE launch (Sec. 4 "Build": the pass at the prefill-decode
 * boundary summarises the whole prompt, every layer of it).  All layers share kv's geometry (strides, block table,
 * lengths, page ranges); layer l reads its keys from k_layers[l] (kv->k is ignored) and writes summaries_layers[l].
 * k_layers and summaries_layers are DEVICE arrays of num_layers device pointers (the caller's; read by the kernel,
 * so they must stay valid until the launch has run); 1 <= num_layers, batch * num_layers <= 65535.  Each summary is
 * byte-identical to what locks_build_summaries writes for that layer alone. */
int locks_build_summaries_layers(locks_ctx *ctx, const locks_kv *kv, const void *const *k_layers,
                                 void *const *summaries_layers, int num_layers, int batch, const int32_t *page_begin,
                                 const int32_t *page_end, locks_stream stream);

/* ---- Page-sharded decode -------------------------------------------------------------------------------------
 * One long request (the GLM-shaped 128K..1M case) whose pages are dealt to several GPUs in page order.  The path
 * itself has no exchange step (every (request, KV head) owns its pages); sharding ONE sequence adds three small
 * ones, which the caller runs with its own collective (torch.distributed / NCCL all-gather of a few KB):
 *   (1) the per-head partition functions log Z_g of the shards, (2) each shard's top-(k-2) candidates (key, page),
 *   (3) each shard's attention partial (out, lse).
 * A shard is presented to the library as an ordinary sequence: [sink or a dummy page] + its candidate pages + [the
 * request's last page or a dummy page], so that "pages 1 .. P-2 are the candidates" holds shard by shard.
 *
 * locks_scan: Eq. 1 over the shard's pages (as locks_select does), plus head_logz [batch][Hq] = log sum over the
 * shard's candidate pages of exp s^_j(q_g) (-inf if it has none).  page_logmass optional (else kept in the
 * workspace for locks_select_scored). */
int locks_scan(locks_ctx *ctx, const void *q, const void *summaries, const locks_kv *kv, int batch, float *page_logmass,
               float *head_logz, locks_stream stream);
/* The selection of locks_select on scores that are already there, with the partition functions given from
 * outside: head_logz_parts [nparts][batch][Hq] (every shard's locks_scan output, gathered); log Z_g = log sum of
 * their exponentials.  page_logmass NULL: the scores the last locks_scan of this context left in the workspace.
 * Outputs as locks_select (the shard's own table and keys); needs more than k pages in the shard. */
int locks_select_scored(locks_ctx *ctx, const float *page_logmass, const float *head_logz_parts, int nparts,
                        const locks_kv *kv, int batch, int32_t *page_ids, int32_t *page_count, float *page_logshare,
                        locks_stream stream);
/* Global top-(k-2) of the shards' candidate lists: cand_key / cand_page [nparts][batch][Hkv][k-2] (ranking key and
 * GLOBAL logical page of each shard's winners, in page order, shards in page order; page -1 = empty slot) ->
 * page_ids [batch][Hkv][k-2] global pages ascending, -1 padded; page_count [batch][Hkv].  Ties to the lower page. */
int locks_merge_selection(locks_ctx *ctx, const float *cand_key, const int32_t *cand_page, int nparts, int batch,
                          int32_t *page_ids, int32_t *page_count, locks_stream stream);
/* Merge of the shards' attention partials (each locks_sparse_attend output normalised over the shard's own pages,
 * with its lse): part_out [nparts][batch][Hq][d] (q dtype), part_lse [nparts][batch][Hq] (-inf: the shard attended
 * nothing) -> out [batch][Hq][d], lse optional. */
int locks_merge_attention(locks_ctx *ctx, const void *part_out, const float *part_lse, int nparts, int batch, void *out,
                          float *lse, locks_stream stream);

/* KV-cache quantisation stacked on the selector (Sec. 5 "KV-cache quantization under extreme sparsity"; App. C,
 * KIVI x LOCKS grid): fake-quantise (quantise, then dequantise in the cache's own element type, in place) every
 * COMPLETE page p with page_begin[b] <= p < page_end[b] (NULL, NULL: all complete pages) of every request and KV
 * head.  KIVI's grouping, page-aligned as in the paper's protocol: keys per channel over the 16 tokens of the page,
 * values per token over groups of 32 consecutive dimensions; asymmetric uniform grid of 2^bits levels between a
 * group's minimum and maximum (bits 1..8; the paper measures 4 and 2).  The partial last page is left untouched
 * (the paper keeps it unquantised inside the always-attended window).  The two arms of the paper's grid are call
 * orders: "post" = locks_build_summaries, then this; "pre" = this, then locks_build_summaries.  Attention and
 * scoring then run unchanged on the quantised values. */
int locks_fake_quantize_pages(locks_ctx *ctx, const locks_kv *kv, int batch, const int32_t *page_begin,
                              const int32_t *page_end, int bits, locks_stream stream);

/* Stage A, "score-then-select" (Sec. 4 "Score (every step)", Eq. 1; share-average combine;
 * App. E): for every request and query head, s^_j(q_g) for all pages j <= P-2 from the resident
 * summaries; shares normalised over the candidates 1..P-2; m_bar_j = mean over the group; per KV
 * head keep page 0, page P-1 and the top k-2 candidates by log m_bar_j (ties: lower index).
 * P <= k keeps every page.
 *   q            [batch][Hq][d] (q_dtype)
 *   page_ids     [batch][Hkv][k] int32 logical page ids, ascending, -1 padded
 *   page_count   [batch][Hkv] int32
 *   page_logmass  optional [batch][Hq][max_pages_per_seq] fp32: s^ for pages 0..P-2 (rest untouched)
 *   page_logshare optional [batch][Hkv][max_pages_per_seq] fp32: log m_bar_j for pages 1..P-2
 * seq_lens[b] = T_b. */
int locks_select(locks_ctx *ctx, const void *q, const void *summaries, const locks_kv *kv, int batch,
                 int32_t *page_ids, int32_t *page_count, float *page_logmass, float *page_logshare,
                 locks_stream stream);

/* The exact-LSE arm (Lemma 1(ii); the "Oracle" / "exact LSE (ceiling)" rows of the paper's tables): the same
 * selection as locks_select, but ranked by the exact page log-mass s_j(q_g) = log sum_{i in P_j} exp(q_g.k_i/sqrt(d))
 * computed from the K pages themselves (reads 4 KB per (page, KV head): a diagnostic, not the hot path).  Same
 * share-average combine, candidates, tie rule and outputs as locks_select, except that page_logmass (optional,
 * [batch][Hq][max_pages_per_seq]) receives the exact mass of ALL pages 0..P-1 (the last page over its valid
 * tokens), which locks_selection_quality needs. */
int locks_select_exact(locks_ctx *ctx, const void *q, const locks_kv *kv, int batch, int32_t *page_ids,
                       int32_t *page_count, float *page_logmass, float *page_logshare, locks_stream stream);

/* Rival page scorers the paper measures the summary against (App. B selection-fidelity table; Sec. 2 / App. A),
 * run through the SAME combine and selection as locks_select, for diagnostics:
 *   LOCKS_SCORER_CENTROID  q.mu_j/sqrt(d) + log B: the centroid term of Eq. 1 alone (from the stored summary);
 *   LOCKS_SCORER_MOMENT    the rank-r moment core, Eq. 3: q.mu_j/sqrt(d) + log B + (1/(2 B d)) sum_{l<=r} sigma_l^2
 *                          (v_l.q)^2, i.e. the second-cumulant truncation of the page mass, computed from the
 *                          stored summary as (1/(2B)) sum_i z_i^2 with z_i the reconstructed within-page logits;
 *   LOCKS_SCORER_ENVELOPE  the min/max envelope (Quest), Lemma 2: sum_c max(q_c u_jc, q_c l_jc)/sqrt(d) with the
 *                          per-dimension key extremes u, l of the page, computed from the K pages (`summaries`
 *                          may be NULL).
 * page_score (optional) [batch][Hq][max_pages_per_seq]: the rival's score of pages 0..P-2 (envelope: 0..P-1);
 * page_logshare (optional): its ranking key.  Plain fp32 kernels: a measuring device, not a fast path. */
#define LOCKS_SCORER_SUMMARY 0
#define LOCKS_SCORER_CENTROID 1
#define LOCKS_SCORER_MOMENT 2
#define LOCKS_SCORER_ENVELOPE 3
int locks_select_rival(locks_ctx *ctx, int scorer, const void *q, const void *summaries, const locks_kv *kv, int batch,
                       int32_t *page_ids, int32_t *page_count, float *page_score, float *page_logshare,
                       locks_stream stream);

/* Selection fidelity of a page table against exact masses (the paper's App. B "microscope" metrics), per
 * (request, KV head), means over the heads of the group:
 *   quality[(b*Hkv + h)*4 + 0] = gamma    total attention mass captured:  sum_{j in S} e^{s_j} / sum_{j<P} e^{s_j}
 *                         + 1] = gamma_c  contested mass: pages 0 and P-1 (always kept) taken out of numerator and
 *                                         denominator
 *                         + 2] = recall   overlap of the candidate pages of S with those of the reference table
 *                         + 3] = needle   of the marked pages the reference table keeps, the fraction S keeps too
 *   exact_logmass [batch][Hq][max_pages_per_seq] from locks_select_exact; (page_ids, page_count) the table under
 *   test; (ref_ids, ref_count) the reference (locks_select_exact's); marked_pages [batch][n_marked] logical pages
 *   (-1 = unused slot) or NULL with n_marked = 0 (needle then reads 1).  An empty denominator reads 1. */
int locks_selection_quality(locks_ctx *ctx, const float *exact_logmass, const locks_kv *kv, int batch,
                            const int32_t *page_ids, const int32_t *page_count, const int32_t *ref_ids,
                            const int32_t *ref_count, const int32_t *marked_pages, int n_marked, float *quality,
                            locks_stream stream);

/* Stage B, sparse paged attention (Sec. 3 "Decode-time attention"; App. E): for every query head,
 * softmax(q.k_i/sqrt(d))-weighted mean of v_i over the tokens i < T_b of the listed pages
 * (split over CTAs, partial results merged by log-sum-exp).  page_ids == NULL: every page, i.e.
 * dense flash-decode over the whole cache (the dense baseline).
 *   out [batch][Hq][d] (q_dtype), lse optional [batch][Hq] fp32 (natural log). */
int locks_sparse_attend(locks_ctx *ctx, const void *q, const locks_kv *kv, int batch,
                        const int32_t *page_ids, const int32_t *page_count, void *out, float *lse,
                        locks_stream stream);

/* One fused decode step for one attention layer (App. E, Fig. 5), legal under stream capture:
 *   1. if k_new != NULL: write k_new/v_new [batch][Hkv][d] at position seq_lens[b] of each
 *      sequence and increment seq_lens[b] (so afterwards seq_lens[b] = T_b counts the new token);
 *      if k_new == NULL the cache and seq_lens already include the token being decoded;
 *   2. locks_select on the resident summaries;  3. locks_sparse_attend on the selected pages;
 *   4. if a page became complete at this step (T_b % B == 0) build its summary, so that it is a
 *      candidate from the next step on (the newly written token is never scored, App. E(i)).
 * These are the results; inside, the token is counted from the first kernel on, its rows are written by
 * the selector's kernel (no page summary depends on them) and seq_lens is stored back there, so the
 * append costs no launch of its own.  k_new / v_new: device, 16-byte aligned.  A sequence whose
 * block-table row is full keeps its length, nothing is written for it and LOCKS_ERR_BAD_BLOCK is
 * recorded in the status word.
 * page_ids / page_count may be NULL (kept in the workspace). */
int locks_decode_step(locks_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                      locks_kv *kv, void *summaries, int batch, void *out, int32_t *page_ids,
                      int32_t *page_count, locks_stream stream);

/* The same step for a caller whose per-step tensors live in HOST memory (pinned for the copies
 * to be asynchronous): copies q_host (and k_new_host / v_new_host if given) to staging space in
 * the workspace, runs locks_decode_step, copies out back to out_host (and the page ids / counts
 * if page_ids_host / page_count_host are given) and synchronises the stream before returning.
 * The cache, summaries, block table and seq_lens stay on the device.
 * Host buffers that the device can address (page-locked and mapped, as cudaHostAlloc returns them) are not
 * copied by the copy engine: one small kernel fetches q / k_new / v_new over the bus and the attention kernel
 * writes out_host itself, which saves four copy nodes per step; other buffers go through async copies.
 * Repeated calls with the same arguments (a serving loop calls once per layer and step with fixed
 * buffers) are cached: from the third call on, the copies and the step are one CUDA-graph launch.
 * The cache holds 8 argument sets per context, needs page-locked host buffers and a stream that is
 * not being captured, and is released by locks_destroy(); other calls take the plain path.
 * LIFETIME: a cached graph holds the device's alias of the page-locked host buffers and every device pointer
 * of the argument set.  Buffers passed to this call must therefore stay allocated and page-locked until
 * locks_destroy() or locks_host_cache_clear(): a later call with the same addresses replays the graph without
 * looking at the memory behind them again.  Call locks_host_cache_clear() before freeing or unpinning any of
 * them if the context lives on. */
int locks_decode_step_host(locks_ctx *ctx, const void *q_host, const void *k_new_host,
                           const void *v_new_host, locks_kv *kv, void *summaries, int batch,
                           void *out_host, int32_t *page_ids_host, int32_t *page_count_host,
                           locks_stream stream);

/* Drop every cached graph of locks_decode_step_host (see its LIFETIME note).  The next calls take the plain
 * path and rebuild the cache from the buffers they are given.  Host-side only. */
int locks_host_cache_clear(locks_ctx *ctx);

/* Copy the sticky device status word to the host and clear it.  Synchronises the stream.
 * *status_host: LOCKS_OK or the first LOCKS_ERR_* a kernel recorded. */
int locks_poll_status(locks_ctx *ctx, int32_t *status_host, locks_stream stream);

/* How the scan (Eq. 1 over every candidate page of every request) deals the pages of a batch to its warps.
 * The scores do not depend on it; log Z is summed in a different order (rounding only).
 *   LOCKS_PARTITION_STRIDED   a fixed share of the warps per (request, KV head): best when the sequences
 *                             are about equally long;
 *   LOCKS_PARTITION_BALANCED  equally many pages per warp, whatever the mix of lengths;
 *   LOCKS_PARTITION_AUTO      (default) every locks_decode_step leaves, in a page-locked word, a suggestion
 *                             for the lengths it saw; the next call that scans follows it.  A captured CUDA
 *                             graph keeps the choice made at capture time.
 * Host-side setting, takes effect from the next call.  LOCKS_ERR_INVALID_ARG for an unknown mode. */
#define LOCKS_PARTITION_AUTO 0
#define LOCKS_PARTITION_STRIDED 1
#define LOCKS_PARTITION_BALANCED 2
int locks_set_scan_partition(locks_ctx *ctx, int mode);
/* The partition the most recent scan launch of this context used (LOCKS_PARTITION_STRIDED or _BALANCED; 0 before
 * the first one, or when the scan ran the plain kernel that has no partition).  With LOCKS_PARTITION_AUTO the
 * choice follows a word the device writes asynchronously, so it can differ from run to run near the switching
 * point; a captured graph (the host entry point's cached graphs included) keeps the choice made at capture.
 * Callers that need reproducible log Z rounding or timings pin the mode with locks_set_scan_partition(), which
 * also drops the host entry point's cached graphs when the mode changes. */
int locks_last_scan_partition(const locks_ctx *ctx);

/* Self-test of the bounded device-side wait every kernel of the library uses for its asynchronous copies: one
 * warp waits, for at most limit_ms milliseconds (1 .. 1000), on a barrier that nothing ever completes, gives up,
 * and records LOCKS_ERR_TIMEOUT in the status word, which locks_poll_status() then reports.  The context stays
 * usable.  Enqueues one small kernel on `stream`. */
int locks_selftest_wait_timeout(locks_ctx *ctx, int limit_ms, locks_stream stream);

/* Number of kernels the last call on this context enqueued (for launch accounting). */
int locks_last_launch_count(const locks_ctx *ctx);

/* Per-stage timing of eager (not captured) locks_decode_step calls, the event-pair split of the
 * step asked for when reporting where the time goes (the paper reports none per kernel).  After
 * locks_profile_begin(ctx, max_steps) every locks_decode_step records CUDA events on its stream at
 * the stage boundaries; locks_profile_end() synchronises the device, writes the mean duration in
 * milliseconds of {summary scan, selection (with the append), sparse attention} to stage_ms[3], the
 * number of steps seen to *steps, and releases the events. */
int locks_profile_begin(locks_ctx *ctx, int max_steps);
int locks_profile_end(locks_ctx *ctx, float *stage_ms, int *steps);
/* A locks_decode_step CAPTURED while profiling is on records the same stage boundaries as event
 * nodes of the graph (always into the first slot).  After a replay, locks_profile_read()
 * synchronises `stream` and writes that replay's three stage durations (ms) to stage_ms[3]. */
int locks_profile_read(locks_ctx *ctx, float *stage_ms, locks_stream stream);

/* locks_sparse_attend for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a convenience of the library).  Some hosts of this code may not call
 * cudaMalloc at all: a plugin running inside an engine that has already handed the whole device to
 * its own memory pool, code on a latency-critical path where an allocation (an implicit device
 * synchronisation) is not acceptable, or a process whose memory budget is fixed up front.  Such a
 * caller cannot provide the workspace locks_create() asks for, so this entry point needs neither a
 * context nor a workspace: the split partials and the split-arrival counters live in an array that is
 * part of the library itself (about 2.1 MB, resident on every GPU that loads the library until the
 * process exits).  Inputs and outputs are the caller's, exactly as for locks_sparse_attend; `cfg`
 * supplies the shapes (head counts, max_pages_per_seq = row length of block_table, budget_tokens =
 * row length * page_size of page_ids, sm_scale).  bf16 only.
 *  - Limit: batch * num_q_heads <= LOCKS_NOALLOC_MAX_ROWS, at most LOCKS_NOALLOC_MAX_SPLITS splits
 *    per KV head; a larger problem is refused with LOCKS_ERR_TOO_LARGE before anything is launched.
 *  - The first call on each device looks up the array's address on that device and sets kernel
 *    attributes; make that first call outside any stream capture, with the device current.
 *  - All calls share the one array, which keeps what the previous call left behind; each call
 *    clears the counters it needs on `stream` first.  Two calls that overlap on the GPU (different
 *    streams, or different host threads) race on it: serialise them.
 *  - No cudaMalloc / cudaFree or allocating library routine is called, here or in the kernel.
 * Device-detected bad page or block ids are skipped as usual but cannot be polled from here. */
#define LOCKS_NOALLOC_MAX_ROWS 256
#define LOCKS_NOALLOC_MAX_SPLITS 16
int locks_sparse_attend_noalloc(const locks_config *cfg, const void *q, const locks_kv *kv, int batch,
                                const int32_t *page_ids, const int32_t *page_count, void *out, float *lse,
                                locks_stream stream);

const char *locks_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* LOCKS_H_ */
