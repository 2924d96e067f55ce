// C-ABI entry points of liblocks (see include/locks.h for the contract of every call).
#include <mutex>
#include <new>

#include "locks_internal.cuh"

namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int validate(const locks_config *c) {
  if (!c) return LOCKS_ERR_INVALID_ARG;
  if (c->num_q_heads <= 0 || c->num_kv_heads <= 0 || c->num_q_heads % c->num_kv_heads) return LOCKS_ERR_INVALID_ARG;
  if (c->max_batch <= 0 || c->max_pages_per_seq <= 0 || c->rank <= 0) return LOCKS_ERR_INVALID_ARG;
  if (c->page_size <= 0 || c->head_dim <= 0) return LOCKS_ERR_INVALID_ARG;
  const int k = (c->budget_tokens + c->page_size - 1) / c->page_size;
  if (c->budget_tokens <= 0 || k < 2) return LOCKS_ERR_INVALID_ARG;
  if (!(c->sm_scale > 0.f)) return LOCKS_ERR_INVALID_ARG;
  if (c->summary_fmt < LOCKS_FMT_F32 || c->summary_fmt > LOCKS_FMT_BF16) return LOCKS_ERR_INVALID_ARG;
  if (c->combine < LOCKS_COMBINE_SHARE_AVG || c->combine > LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_INVALID_ARG;
  if ((c->kv_dtype != LOCKS_F32 && c->kv_dtype != LOCKS_BF16) || (c->q_dtype != LOCKS_F32 && c->q_dtype != LOCKS_BF16))
    return LOCKS_ERR_INVALID_ARG;
  if (c->head_dim != LOCKS_D) return LOCKS_ERR_UNSUPPORTED;
  // pages of 32 and 64 tokens (App. D "Page size") run on the plain fp32 kernels
  if (c->page_size != LOCKS_B && c->page_size != 32 && c->page_size != 64) return LOCKS_ERR_UNSUPPORTED;
  if (c->num_q_heads / c->num_kv_heads > 16) return LOCKS_ERR_UNSUPPORTED;
  if (c->kv_dtype != c->q_dtype) return LOCKS_ERR_UNSUPPORTED;
  if (c->summary_fmt == LOCKS_FMT_I4 && c->rank != 2 && c->rank != 4 && c->rank != 8) return LOCKS_ERR_UNSUPPORTED;
  if (c->summary_fmt != LOCKS_FMT_I4 && c->rank > 16) return LOCKS_ERR_UNSUPPORTED;
  const int chunk_max = LOCKS_SEL_THREADS * LOCKS_SEL_MAX_EPT;
  const int chunks = (c->max_pages_per_seq + chunk_max - 1) / chunk_max;
  if (chunks > 1 && (size_t)chunks * (k - 2) > 16 * LOCKS_SEL_THREADS) return LOCKS_ERR_UNSUPPORTED;
  if (k > LOCKS_SEL_THREADS * 4) return LOCKS_ERR_UNSUPPORTED;
  return LOCKS_OK;
}

struct Layout {
  size_t status, shat, part, part_cnt, sel_done, cand_val, cand_idx, att_o, att_lse, att_done, ids, cnt, sq, skn, svn, sout, seq_eff, total;
  int G, k, S, max_groups, sel_ept, sel_chunks, sel_kc;
};

Layout make_layout(const locks_config *c) {
  Layout L;
  L.G = c->num_q_heads / c->num_kv_heads;
  L.k = (c->budget_tokens + c->page_size - 1) / c->page_size;
  L.S = locks_fmt_stride(c->summary_fmt, c->rank, c->page_size);
  L.max_groups = (c->max_pages_per_seq + LOCKS_GROUP - 1) / LOCKS_GROUP;
  // Pages per thread of a selector CTA (1 .. 16; a CTA ranks sel_ept * 512 pages).  With many (request,
  // KV head) problems and a context of up to 8192 pages, one CTA ranks a whole problem.  Otherwise a problem is
  // cut into chunks whose top-(k-2) lists are ranked by the chunk that arrives last, and the chunk size is the
  // one a small cost model likes best (microseconds, fitted to measurements on B200 at 2 .. 256 problems,
  // G = 4 .. 16, 8K .. 64K pages): a CTA's chain of round trips costs about 6 plus 1.2 per batch of 16 score
  // loads per thread beyond the first one and a half, plus 0.15 per 512 pages; the CTAs of a launch run in
  // waves of one per SM; the final ranking costs 3.3 plus 0.43 per 512 candidates.
  const int per_thread = (c->max_pages_per_seq + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS;
  // (per-head arm: one ranking per query head)
  const int64_t problems = (int64_t)c->max_batch * (c->combine == LOCKS_COMBINE_PER_HEAD ? c->num_q_heads : c->num_kv_heads);
  const int kcand = L.k - 2 > 0 ? L.k - 2 : 1;
  L.sel_ept = LOCKS_SEL_MAX_EPT;
  if (problems >= 32 && per_thread <= LOCKS_SEL_MAX_EPT) {
    L.sel_ept = per_thread;
  } else {
    constexpr int kSms = 148;   // the model's machine; the layout must not depend on the device at hand
    double best = 1e30;
    for (int ept = 1; ept <= LOCKS_SEL_MAX_EPT; ept *= 2) {
      const int chunks = (c->max_pages_per_seq + ept * LOCKS_SEL_THREADS - 1) / (ept * LOCKS_SEL_THREADS);
      if (chunks > 1 && (size_t)chunks * kcand > (size_t)LOCKS_SEL_MAX_EPT * LOCKS_SEL_THREADS) continue;
      const double batches = (double)ept * L.G / 16.0;
      const double cta = 6.0 + 1.2 * (batches > 1.5 ? batches - 1.5 : 0.0) + 0.15 * ept;
      const double waves = (double)((problems * chunks + kSms - 1) / kSms);
      const double fin = chunks == 1 ? 0.0 : 3.3 + 0.43 * (double)chunks * kcand / LOCKS_SEL_THREADS;
      const double est = waves * cta + fin;
      if (est < best) {
        best = est;
        L.sel_ept = ept;
      }
      if (chunks == 1) break;
    }
  }
  L.sel_chunks = (c->max_pages_per_seq + L.sel_ept * LOCKS_SEL_THREADS - 1) / (L.sel_ept * LOCKS_SEL_THREADS);
  L.sel_kc = L.k - 2 > 0 ? L.k - 2 : 1;
  const size_t nb = c->max_batch, Hq = c->num_q_heads, Hkv = c->num_kv_heads, P = c->max_pages_per_seq;
  const size_t esz = c->q_dtype == LOCKS_BF16 ? 2 : 4;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  L.status = take(64);
  L.shat = take(nb * Hq * P * 4);
  L.part = take(nb * Hq * L.max_groups * 8);
  L.part_cnt = take(nb * Hkv * 4);
  const size_t Hsel = c->combine == LOCKS_COMBINE_PER_HEAD ? Hq : Hkv;   // rankings per request
  L.sel_done = take(nb * Hq * 4);
  L.cand_val = take(nb * Hsel * L.sel_chunks * L.sel_kc * 4);
  L.cand_idx = take(nb * Hsel * L.sel_chunks * L.sel_kc * 4);
  // split-K partial rows: batch * Hq * splits with splits <= slots / (batch * Hkv) (+1 rounding) and <= 128
  const size_t att_rows = (size_t)L.G * LOCKS_ATT_SLOT_BOUND + 2 * nb * Hq;
  L.att_o = take(att_rows * LOCKS_D * 4);
  L.att_lse = take(att_rows * 4);
  L.att_done = take(nb * Hq * 4);
  L.ids = take(nb * Hsel * L.k * 4);
  L.cnt = take(nb * Hsel * 4);
  L.sq = take(nb * Hq * LOCKS_D * esz);
  L.skn = take(nb * Hkv * LOCKS_D * esz);
  L.svn = take(nb * Hkv * LOCKS_D * esz);
  L.sout = take(nb * Hq * LOCKS_D * esz);
  L.seq_eff = take(2 * nb * 4);
  L.total = o;
  return L;
}

int check_common(const locks_ctx *ctx, const locks_kv *kv, int batch) {
  if (!ctx || !kv || !kv->k || !kv->v || !kv->block_table || !kv->seq_lens) return LOCKS_ERR_INVALID_ARG;
  if (batch <= 0 || batch > ctx->cfg.max_batch || kv->num_blocks <= 0) return LOCKS_ERR_INVALID_ARG;
  if (kv->stride_block <= 0 || kv->stride_head <= 0 || kv->stride_token < LOCKS_D) return LOCKS_ERR_INVALID_ARG;
  // 16-byte vector copies of cache rows
  if ((kv->stride_block | kv->stride_head | kv->stride_token) % (ctx->cfg.kv_dtype == LOCKS_BF16 ? 8 : 4))
    return LOCKS_ERR_INVALID_ARG;
  if (((uintptr_t)kv->k | (uintptr_t)kv->v) % 16) return LOCKS_ERR_INVALID_ARG;
  return LOCKS_OK;
}

}  // namespace

bool locks_attrs_needed(int family) {
  static std::mutex mu;
  static uint64_t done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || family < 0 || family >= 64) return true;
  std::lock_guard<std::mutex> lock(mu);
  const uint64_t bit = 1ull << family;
  if (done[dev] & bit) return false;
  done[dev] |= bit;
  return true;
}

extern "C" {

size_t locks_summary_bytes(const locks_config *cfg) {
  if (validate(cfg) != LOCKS_OK) return 0;
  return (size_t)make_layout(cfg).S;
}

size_t locks_workspace_bytes(const locks_config *cfg) {
  if (validate(cfg) != LOCKS_OK) return 0;
  return make_layout(cfg).total;
}

int locks_create(const locks_config *cfg, void *workspace, size_t ws_bytes, locks_ctx **out) {
  if (!out) return LOCKS_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate(cfg);
  if (rc != LOCKS_OK) return rc;
  const Layout L = make_layout(cfg);
  if (!workspace || ws_bytes < L.total || ((uintptr_t)workspace % 256)) return LOCKS_ERR_WORKSPACE;
  locks_ctx *c = new (std::nothrow) locks_ctx();
  if (!c) return LOCKS_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->prof_ev = nullptr; c->prof_cap = c->prof_n = 0;
  c->att_cluster_max = -1;
  for (int i = 0; i < LOCKS_HOST_GRAPHS; ++i) c->hg[i] = locks_host_graph{};
  c->hg_next = 0;
  c->part_slots = L.max_groups;
  c->part_balanced = 0;
  c->scan_partition = LOCKS_PARTITION_AUTO;
  c->last_partition = 0;
  c->scorer = LOCKS_SCORER_SUMMARY;
  c->hint_host = nullptr; c->hint_dev = nullptr;
  {   // one page-locked word the device can write and the host can read without synchronising
    void *hp = nullptr, *dp = nullptr;
    if (cudaHostAlloc(&hp, 64, cudaHostAllocMapped) == cudaSuccess) {
      if (cudaHostGetDevicePointer(&dp, hp, 0) == cudaSuccess) {
        c->hint_host = reinterpret_cast<int32_t *>(hp);
        c->hint_dev = reinterpret_cast<int32_t *>(dp);
        *c->hint_host = 0;
      } else {
        cudaFreeHost(hp);
      }
    }
    (void)cudaGetLastError();   // without the word the partition simply stays strided
  }
  c->G = L.G; c->k = L.k; c->S = L.S; c->Pmax = cfg->max_pages_per_seq; c->max_groups = L.max_groups;
  c->B = cfg->page_size;
  c->sel_ept = L.sel_ept; c->sel_chunks = L.sel_chunks; c->sel_kc = L.sel_kc;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    if (c->hint_host) cudaFreeHost(c->hint_host);
    delete c;
    return LOCKS_ERR_CUDA;
  }
  char *ws = reinterpret_cast<char *>(workspace);
  c->ws = ws; c->ws_bytes = ws_bytes;
  c->status = reinterpret_cast<int32_t *>(ws + L.status);
  c->shat = reinterpret_cast<float *>(ws + L.shat);
  c->part = reinterpret_cast<float2 *>(ws + L.part);
  c->part_cnt = reinterpret_cast<int32_t *>(ws + L.part_cnt);
  c->sel_done = reinterpret_cast<int32_t *>(ws + L.sel_done);
  c->cand_val = reinterpret_cast<float *>(ws + L.cand_val);
  c->cand_idx = reinterpret_cast<int32_t *>(ws + L.cand_idx);
  c->att_o = reinterpret_cast<float *>(ws + L.att_o);
  c->att_lse = reinterpret_cast<float *>(ws + L.att_lse);
  c->att_done = reinterpret_cast<int32_t *>(ws + L.att_done);
  c->ids_int = reinterpret_cast<int32_t *>(ws + L.ids);
  c->cnt_int = reinterpret_cast<int32_t *>(ws + L.cnt);
  c->seq_eff = reinterpret_cast<int32_t *>(ws + L.seq_eff);
  c->stage_q = ws + L.sq; c->stage_kn = ws + L.skn; c->stage_vn = ws + L.svn; c->stage_out = ws + L.sout;
  if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
      cudaMemsetAsync(c->status, 0, 64, 0) != cudaSuccess ||
      cudaMemsetAsync(c->att_done, 0, (size_t)cfg->max_batch * cfg->num_q_heads * 4, 0) != cudaSuccess ||
      cudaMemsetAsync(c->sel_done, 0, (size_t)cfg->max_batch * cfg->num_q_heads * 4, 0) != cudaSuccess ||
      cudaMemsetAsync(c->part_cnt, 0, (size_t)cfg->max_batch * cfg->num_kv_heads * 4, 0) != cudaSuccess ||
      cudaStreamSynchronize(0) != cudaSuccess) {
    if (c->hint_host) cudaFreeHost(c->hint_host);
    delete c;
    return LOCKS_ERR_CUDA;
  }
  *out = c;
  return LOCKS_OK;
}

int locks_destroy(locks_ctx *ctx) {
  if (!ctx) return LOCKS_ERR_INVALID_ARG;
  if (ctx->prof_ev) {
    for (int i = 0; i < ctx->prof_cap * LOCKS_PROF_MARKS; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    delete[] ctx->prof_ev;
  }
  for (int i = 0; i < LOCKS_HOST_GRAPHS; ++i)
    if (ctx->hg[i].exec) cudaGraphExecDestroy(ctx->hg[i].exec);
  cudaEventDestroy(ctx->ev_fork);
  cudaEventDestroy(ctx->ev_join);
  cudaStreamDestroy(ctx->side);
  if (ctx->hint_host) cudaFreeHost(ctx->hint_host);
  delete ctx;
  return LOCKS_OK;
}

namespace {
__global__ void __launch_bounds__(32) wait_timeout_kernel(int32_t *status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncwarp();
  if (!mbar_wait(&bar, 0, limit_ns) && threadIdx.x == 0) set_status(status, LOCKS_ERR_TIMEOUT);
}
}  // namespace

int locks_selftest_wait_timeout(locks_ctx *ctx, int limit_ms, locks_stream stream) {
  if (!ctx || limit_ms < 1 || limit_ms > 1000) return LOCKS_ERR_INVALID_ARG;
  wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->status, (uint64_t)limit_ms * 1000000ull);
  return cudaPeekAtLastError() == cudaSuccess ? LOCKS_OK : LOCKS_ERR_CUDA;
}

int locks_set_scan_partition(locks_ctx *ctx, int mode) {
  if (!ctx || mode < LOCKS_PARTITION_AUTO || mode > LOCKS_PARTITION_BALANCED) return LOCKS_ERR_INVALID_ARG;
  if (mode != ctx->scan_partition) (void)locks_host_cache_clear(ctx);   // cached graphs froze the old choice
  ctx->scan_partition = mode;
  return LOCKS_OK;
}

int locks_last_scan_partition(const locks_ctx *ctx) { return ctx ? ctx->last_partition : 0; }

int locks_host_cache_clear(locks_ctx *ctx) {
  if (!ctx) return LOCKS_ERR_INVALID_ARG;
  for (int i = 0; i < LOCKS_HOST_GRAPHS; ++i) {
    if (ctx->hg[i].exec) cudaGraphExecDestroy(ctx->hg[i].exec);
    ctx->hg[i] = locks_host_graph{};
  }
  ctx->hg_next = 0;
  return LOCKS_OK;
}

int locks_build_summaries(locks_ctx *ctx, const locks_kv *kv, int batch, const int32_t *page_begin,
                          const int32_t *page_end, void *summaries, locks_stream stream) {
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!summaries || ((uintptr_t)summaries % 16) || ((page_begin == nullptr) != (page_end == nullptr)))
    return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_build(ctx, kv, batch, page_begin, page_end, 0, summaries, nullptr, nullptr, (cudaStream_t)stream);
}

int locks_build_summaries_layers(locks_ctx *ctx, const locks_kv *kv, const void *const *k_layers,
                                 void *const *summaries_layers, int num_layers, int batch, const int32_t *page_begin,
                                 const int32_t *page_end, locks_stream stream) {
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  if (!kv || !k_layers || !summaries_layers || num_layers < 1) return LOCKS_ERR_INVALID_ARG;
  locks_kv kv0 = *kv;
  // kv->k and kv->v are not read by this call: a placeholder passes the common checks
  kv0.k = reinterpret_cast<void *>(uintptr_t(256));
  kv0.v = kv0.k;
  int rc = check_common(ctx, &kv0, batch);
  if (rc != LOCKS_OK) return rc;
  if ((int64_t)batch * num_layers > 65535 || ((page_begin == nullptr) != (page_end == nullptr))) return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_build(ctx, &kv0, batch, page_begin, page_end, 0, nullptr, nullptr, nullptr, (cudaStream_t)stream,
                            k_layers, summaries_layers, num_layers);
}

// ---- page-sharded decode: one long request whose pages are dealt to several GPUs (three small exchanges) ------

int locks_scan(locks_ctx *ctx, const void *q, const void *summaries, const locks_kv *kv, int batch, float *page_logmass,
               float *head_logz, locks_stream stream) {
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q || !summaries || !head_logz || ((uintptr_t)summaries % 16) || ((uintptr_t)q % 16)) return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->last_launches = 0;
  if ((rc = locks_launch_scan(ctx, q, summaries, kv, batch, page_logmass ? page_logmass : ctx->shat, 0, st)) != LOCKS_OK) return rc;
  return locks_launch_head_logz(ctx, kv, batch, head_logz, st);
}

int locks_select_scored(locks_ctx *ctx, const float *page_logmass, const float *head_logz_parts, int nparts,
                        const locks_kv *kv, int batch, int32_t *page_ids, int32_t *page_count, float *page_logshare,
                        locks_stream stream) {
  if (ctx && ctx->cfg.combine == LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_UNSUPPORTED;   // one page table per KV head only
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!head_logz_parts || !page_ids || !page_count || nparts < 1) return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->last_launches = 0;
  if ((rc = locks_launch_ext_partials(ctx, head_logz_parts, nparts, batch, st)) != LOCKS_OK) return rc;
  return locks_launch_select(ctx, page_logmass ? page_logmass : ctx->shat, kv, batch, page_ids, page_count, page_logshare,
                             nullptr, st);
}

int locks_merge_selection(locks_ctx *ctx, const float *cand_key, const int32_t *cand_page, int nparts, int batch,
                          int32_t *page_ids, int32_t *page_count, locks_stream stream) {
  if (ctx && ctx->cfg.combine == LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_UNSUPPORTED;   // one page table per KV head only
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  if (!ctx || !cand_key || !cand_page || !page_ids || !page_count || nparts < 1 || batch < 1 || batch > ctx->cfg.max_batch)
    return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_merge_selection(ctx, cand_key, cand_page, nparts, batch, page_ids, page_count, (cudaStream_t)stream);
}

int locks_merge_attention(locks_ctx *ctx, const void *part_out, const float *part_lse, int nparts, int batch, void *out,
                          float *lse, locks_stream stream) {
  if (!ctx || !part_out || !part_lse || !out || nparts < 1 || batch < 1 || batch > ctx->cfg.max_batch)
    return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_merge_shards(ctx, part_out, part_lse, nparts, batch, out, lse, (cudaStream_t)stream);
}

int locks_fake_quantize_pages(locks_ctx *ctx, const locks_kv *kv, int batch, const int32_t *page_begin,
                              const int32_t *page_end, int bits, locks_stream stream) {
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (bits < 1 || bits > 8 || ((page_begin == nullptr) != (page_end == nullptr))) return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_fake_quant(ctx, kv, batch, page_begin, page_end, bits, (cudaStream_t)stream);
}

int locks_select(locks_ctx *ctx, const void *q, const void *summaries, const locks_kv *kv, int batch,
                 int32_t *page_ids, int32_t *page_count, float *page_logmass, float *page_logshare,
                 locks_stream stream) {
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q || !summaries || !page_ids || !page_count || ((uintptr_t)summaries % 16) || ((uintptr_t)q % 16))
    return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->last_launches = 0;
  float *shat = page_logmass ? page_logmass : ctx->shat;
  if ((rc = locks_launch_scan(ctx, q, summaries, kv, batch, shat, 0, st)) != LOCKS_OK) return rc;
  return locks_launch_select(ctx, shat, kv, batch, page_ids, page_count, page_logshare, nullptr, st);
}

int locks_select_exact(locks_ctx *ctx, const void *q, const locks_kv *kv, int batch, int32_t *page_ids,
                       int32_t *page_count, float *page_logmass, float *page_logshare, locks_stream stream) {
  if (ctx && ctx->cfg.combine == LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_UNSUPPORTED;   // one page table per KV head only
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q || !page_ids || !page_count || ((uintptr_t)q % 16)) return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->last_launches = 0;
  float *shat = page_logmass ? page_logmass : ctx->shat;
  if ((rc = locks_launch_exact_scan(ctx, q, kv, batch, shat, 0, st)) != LOCKS_OK) return rc;
  return locks_launch_select(ctx, shat, kv, batch, page_ids, page_count, page_logshare, nullptr, st);
}

int locks_select_rival(locks_ctx *ctx, int scorer, const void *q, const void *summaries, const locks_kv *kv, int batch,
                       int32_t *page_ids, int32_t *page_count, float *page_score, float *page_logshare,
                       locks_stream stream) {
  if (ctx && ctx->cfg.combine == LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_UNSUPPORTED;   // one page table per KV head only
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q || !page_ids || !page_count || ((uintptr_t)q % 16)) return LOCKS_ERR_INVALID_ARG;
  if (scorer != LOCKS_SCORER_CENTROID && scorer != LOCKS_SCORER_MOMENT && scorer != LOCKS_SCORER_ENVELOPE)
    return LOCKS_ERR_INVALID_ARG;
  if (scorer != LOCKS_SCORER_ENVELOPE && (!summaries || ((uintptr_t)summaries % 16))) return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->last_launches = 0;
  float *shat = page_score ? page_score : ctx->shat;
  if (scorer == LOCKS_SCORER_ENVELOPE) {
    rc = locks_launch_exact_scan(ctx, q, kv, batch, shat, 1, st);
  } else {
    ctx->scorer = scorer;
    rc = locks_launch_scan(ctx, q, summaries, kv, batch, shat, 0, st);
    ctx->scorer = LOCKS_SCORER_SUMMARY;
  }
  if (rc != LOCKS_OK) return rc;
  return locks_launch_select(ctx, shat, kv, batch, page_ids, page_count, page_logshare, nullptr, st);
}

int locks_selection_quality(locks_ctx *ctx, const float *exact_logmass, const locks_kv *kv, int batch,
                            const int32_t *page_ids, const int32_t *page_count, const int32_t *ref_ids,
                            const int32_t *ref_count, const int32_t *marked_pages, int n_marked, float *quality,
                            locks_stream stream) {
  if (ctx && ctx->cfg.combine == LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_UNSUPPORTED;   // one page table per KV head only
  if (ctx && ctx->B != LOCKS_B) return LOCKS_ERR_UNSUPPORTED;   // 16-token pages only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!exact_logmass || !page_ids || !page_count || !ref_ids || !ref_count || !quality || n_marked < 0 ||
      (n_marked > 0 && !marked_pages))
    return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_quality(ctx, exact_logmass, kv, batch, page_ids, page_count, ref_ids, ref_count, marked_pages,
                              n_marked, quality, (cudaStream_t)stream);
}

int locks_sparse_attend(locks_ctx *ctx, const void *q, const locks_kv *kv, int batch, const int32_t *page_ids,
                        const int32_t *page_count, void *out, float *lse, locks_stream stream) {
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q || !out || ((page_ids == nullptr) != (page_count == nullptr)) || ((uintptr_t)q % 16))
    return LOCKS_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  return locks_launch_attend(ctx, q, kv, batch, page_ids, page_count, out, lse, (cudaStream_t)stream);
}

int locks_decode_step(locks_ctx *ctx, const void *q, const void *k_new, const void *v_new, locks_kv *kv,
                      void *summaries, int batch, void *out, int32_t *page_ids, int32_t *page_count,
                      locks_stream stream) {
  if (ctx && ctx->cfg.combine == LOCKS_COMBINE_PER_HEAD) return LOCKS_ERR_UNSUPPORTED;   // one page table per KV head only
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q || !summaries || !out || ((k_new == nullptr) != (v_new == nullptr)) || ((uintptr_t)summaries % 16) ||
      ((uintptr_t)q % 16) || ((uintptr_t)k_new % 16) || ((uintptr_t)v_new % 16))
    return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t *ids = page_ids ? page_ids : ctx->ids_int;
  int32_t *cnt = page_count ? page_count : ctx->cnt_int;
  ctx->last_launches = 0;
  cudaEvent_t *pe = (ctx->prof_ev && ctx->prof_n < ctx->prof_cap) ? ctx->prof_ev + ctx->prof_n * LOCKS_PROF_MARKS : nullptr;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (pe) cudaStreamIsCapturing(st, &cap);
  const bool capturing = cap == cudaStreamCaptureStatusActive;
  if (pe && capturing) pe = ctx->prof_ev;   // a captured step always reports through slot 0
  auto mark = [&](int i) {
    if (!pe) return;
    if (capturing) cudaEventRecordWithFlags(pe[i], st, cudaEventRecordExternal);   // becomes an event-record node
    else cudaEventRecord(pe[i], st);
  };
  // The new token is counted from the scan on (lengths one longer, published in the workspace); its K/V
  // rows are written by the selector's kernel, beside the ranking, which is early enough for the two
  // readers of the last page (attention, and the summary build when the token completes a page).
  locks_append app;
  locks_kv kv_step = *kv;
  if (k_new) {
    app.k_new = k_new; app.v_new = v_new; app.k = kv->k; app.v = kv->v;
    app.sb = kv->stride_block; app.sh = kv->stride_head; app.st = kv->stride_token;
    app.block_table = kv->block_table; app.seq_eff = ctx->seq_eff; app.seq_commit = kv->seq_lens;
    app.num_blocks = kv->num_blocks; app.esz = ctx->cfg.kv_dtype == LOCKS_BF16 ? 2 : 4;
    kv_step.seq_lens = ctx->seq_eff;
  }
  mark(0);
  if ((rc = locks_launch_scan(ctx, q, summaries, kv, batch, ctx->shat, k_new ? 1 : 0, st)) != LOCKS_OK) return rc;
  mark(1);
  // The page that this step's token completes (if any) is summarised on a second stream beside the selector
  // and attention: its summary is first read by the next step's scan.  The build starts when the scan has
  // published the lengths; the token itself it takes from k_new, since the selector's kernel is writing it
  // into the cache at the same time.
  if (cudaEventRecord(ctx->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess)
    return LOCKS_ERR_CUDA;
  if ((rc = locks_launch_build(ctx, &kv_step, batch, nullptr, nullptr, 1, summaries, k_new,
                               k_new ? ctx->seq_eff + batch : nullptr, ctx->side)) != LOCKS_OK)
    return rc;
  if (cudaEventRecord(ctx->ev_join, ctx->side) != cudaSuccess) return LOCKS_ERR_CUDA;
  if ((rc = locks_launch_select(ctx, ctx->shat, &kv_step, batch, ids, cnt, nullptr, k_new ? &app : nullptr, st)) != LOCKS_OK)
    return rc;
  mark(2);
  if ((rc = locks_launch_attend(ctx, q, &kv_step, batch, ids, cnt, out, nullptr, st)) != LOCKS_OK) return rc;
  mark(3);
  if (pe && !capturing) ctx->prof_n++;
  if (cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) return LOCKS_ERR_CUDA;
  return LOCKS_OK;
}

namespace {

// The device's address of a page-locked, device-mapped host buffer, or nullptr
void *device_alias(const void *host) {
  if (!host) return nullptr;
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

// q, k_new and v_new fetched over the bus by one kernel, 16 bytes per thread: a copy node per buffer costs
// about 4 us each in a step that lasts under 60
__global__ void __launch_bounds__(256) stage_in_kernel(const uint4 *q, const uint4 *kn, const uint4 *vn, uint4 *dq,
                                                      uint4 *dkn, uint4 *dvn, int nq, int nk) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < nq) dq[i] = q[i];
  else if (i < nq + nk) dkn[i - nq] = kn[i - nq];
  else if (i < nq + 2 * nk) dvn[i - nq - nk] = vn[i - nq - nk];
}

// inputs in, the step, results out -- enqueued on `st` (eagerly, or under capture).  Host buffers that the
// device can address (page-locked and mapped) are read by a staging kernel and written by the attention
// kernel itself; others go through copies.
int enqueue_host_step(locks_ctx *ctx, const void *q_host, const void *k_new_host, const void *v_new_host, locks_kv *kv,
                      void *summaries, int batch, void *out_host, int32_t *page_ids_host, int32_t *page_count_host,
                      cudaStream_t st) {
  const size_t esz = ctx->cfg.q_dtype == LOCKS_BF16 ? 2 : 4;
  const size_t qb = (size_t)batch * ctx->cfg.num_q_heads * LOCKS_D * esz;
  const size_t kb = (size_t)batch * ctx->cfg.num_kv_heads * LOCKS_D * esz;
  auto aligned16 = [](const void *p) { return ((uintptr_t)p % 16) == 0; };
  const void *qa = device_alias(q_host), *ka = device_alias(k_new_host), *va = device_alias(v_new_host);
  void *oa = device_alias(out_host);
  const bool direct_in = qa && aligned16(qa) && (!k_new_host || (ka && va && aligned16(ka) && aligned16(va)));
  int staged = 0;
  if (direct_in) {
    const int nq = (int)(qb / 16), nk = k_new_host ? (int)(kb / 16) : 0;
    stage_in_kernel<<<(nq + 2 * nk + 255) / 256, 256, 0, st>>>(
        reinterpret_cast<const uint4 *>(qa), reinterpret_cast<const uint4 *>(ka), reinterpret_cast<const uint4 *>(va),
        reinterpret_cast<uint4 *>(ctx->stage_q), reinterpret_cast<uint4 *>(ctx->stage_kn),
        reinterpret_cast<uint4 *>(ctx->stage_vn), nq, nk);
    if (cudaPeekAtLastError() != cudaSuccess) return LOCKS_ERR_CUDA;
    staged = 1;
  } else {
    if (cudaMemcpyAsync(ctx->stage_q, q_host, qb, cudaMemcpyHostToDevice, st) != cudaSuccess) return LOCKS_ERR_CUDA;
    if (k_new_host) {
      if (cudaMemcpyAsync(ctx->stage_kn, k_new_host, kb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
          cudaMemcpyAsync(ctx->stage_vn, v_new_host, kb, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return LOCKS_ERR_CUDA;
    }
  }
  const bool direct_out = oa && aligned16(oa);
  int rc = locks_decode_step(ctx, ctx->stage_q, k_new_host ? ctx->stage_kn : nullptr, k_new_host ? ctx->stage_vn : nullptr,
                             kv, summaries, batch, direct_out ? oa : ctx->stage_out, ctx->ids_int, ctx->cnt_int,
                             (locks_stream)st);
  if (rc != LOCKS_OK) return rc;
  ctx->last_launches += staged;
  if (!direct_out && cudaMemcpyAsync(out_host, ctx->stage_out, qb, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return LOCKS_ERR_CUDA;
  if (page_ids_host &&
      cudaMemcpyAsync(page_ids_host, ctx->ids_int, (size_t)batch * ctx->cfg.num_kv_heads * ctx->k * 4,
                      cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return LOCKS_ERR_CUDA;
  if (page_count_host &&
      cudaMemcpyAsync(page_count_host, ctx->cnt_int, (size_t)batch * ctx->cfg.num_kv_heads * 4, cudaMemcpyDeviceToHost,
                      st) != cudaSuccess)
    return LOCKS_ERR_CUDA;
  return LOCKS_OK;
}

bool is_pinned(const void *p) {   // page-locked host memory (or nothing to copy)
  if (!p) return true;
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { (void)cudaGetLastError(); return false; }
  return a.type == cudaMemoryTypeHost;
}

}  // namespace

int locks_decode_step_host(locks_ctx *ctx, const void *q_host, const void *k_new_host, const void *v_new_host,
                           locks_kv *kv, void *summaries, int batch, void *out_host, int32_t *page_ids_host,
                           int32_t *page_count_host, locks_stream stream) {
  int rc = check_common(ctx, kv, batch);
  if (rc != LOCKS_OK) return rc;
  if (!q_host || !out_host || ((k_new_host == nullptr) != (v_new_host == nullptr))) return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  // A caller that repeats the same arguments (one set per layer, every decode step) gets the whole call as
  // one graph launch from the second repetition on: the copies and the four launches cost one submission.
  // Needs page-locked host buffers, a stream that is not being captured, and per-stage timing switched off.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  const bool quiet = cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone && !ctx->prof_ev;
  locks_host_graph *g = nullptr;
  if (quiet) {
    for (int i = 0; i < LOCKS_HOST_GRAPHS && !g; ++i) {
      locks_host_graph &e = ctx->hg[i];
      if (e.seen > 0 && e.q == q_host && e.kn == k_new_host && e.vn == v_new_host && e.out == out_host &&
          e.summ == summaries && e.ids == page_ids_host && e.cnt == page_count_host && e.batch == batch && e.st == st &&
          e.kv.k == kv->k && e.kv.v == kv->v && e.kv.stride_block == kv->stride_block &&
          e.kv.stride_head == kv->stride_head && e.kv.stride_token == kv->stride_token &&
          e.kv.num_blocks == kv->num_blocks && e.kv.block_table == kv->block_table && e.kv.seq_lens == kv->seq_lens)
        g = &e;
    }
  }
  if (g && g->exec) {   // the common case: known arguments (their buffers were page-locked when the entry was made)
    if (cudaGraphLaunch(g->exec, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) return LOCKS_ERR_CUDA;
    ctx->last_launches = g->launches;
    return LOCKS_OK;
  }
  const bool graph_ok = quiet && (g || (is_pinned(q_host) && is_pinned(k_new_host) && is_pinned(v_new_host) &&
                                        is_pinned(out_host) && is_pinned(page_ids_host) && is_pinned(page_count_host)));
  if (graph_ok) {
    if (!g) {   // new arguments: take the next slot
      g = &ctx->hg[ctx->hg_next];
      ctx->hg_next = (ctx->hg_next + 1) % LOCKS_HOST_GRAPHS;
      if (g->exec) cudaGraphExecDestroy(g->exec);
      *g = locks_host_graph{q_host, k_new_host, v_new_host, out_host, summaries, page_ids_host, page_count_host, *kv,
                            batch, st, 0, 0, nullptr};
    }
    if (!g->exec && g->seen >= 1) {   // second call with these arguments: capture
      cudaGraph_t graph = nullptr;
      if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        rc = enqueue_host_step(ctx, q_host, k_new_host, v_new_host, kv, summaries, batch, out_host, page_ids_host,
                               page_count_host, st);
        g->launches = ctx->last_launches;
        const cudaError_t ce = cudaStreamEndCapture(st, &graph);
        if (rc == LOCKS_OK && ce == cudaSuccess && graph) {
          if (cudaGraphInstantiate(&g->exec, graph, 0) != cudaSuccess) g->exec = nullptr;
        }
        if (graph) cudaGraphDestroy(graph);
      }
      (void)cudaGetLastError();   // a failed capture falls back to the eager path below
    }
    if (g->exec) {
      if (cudaGraphLaunch(g->exec, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) return LOCKS_ERR_CUDA;
      ctx->last_launches = g->launches;
      return LOCKS_OK;
    }
    g->seen++;
  }
  rc = enqueue_host_step(ctx, q_host, k_new_host, v_new_host, kv, summaries, batch, out_host, page_ids_host,
                         page_count_host, st);
  if (rc != LOCKS_OK) return rc;
  const int launches = ctx->last_launches;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LOCKS_ERR_CUDA;
  ctx->last_launches = launches;
  return LOCKS_OK;
}

int locks_poll_status(locks_ctx *ctx, int32_t *status_host, locks_stream stream) {
  if (!ctx || !status_host) return LOCKS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(status_host, ctx->status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(ctx->status, 0, 4, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return LOCKS_ERR_CUDA;
  return LOCKS_OK;
}

int locks_last_launch_count(const locks_ctx *ctx) { return ctx ? ctx->last_launches : 0; }

int locks_profile_begin(locks_ctx *ctx, int max_steps) {
  if (!ctx || max_steps <= 0 || ctx->prof_ev) return LOCKS_ERR_INVALID_ARG;
  ctx->prof_ev = new (std::nothrow) cudaEvent_t[(size_t)max_steps * LOCKS_PROF_MARKS];
  if (!ctx->prof_ev) return LOCKS_ERR_INVALID_ARG;
  for (int i = 0; i < max_steps * LOCKS_PROF_MARKS; ++i)
    if (cudaEventCreate(&ctx->prof_ev[i]) != cudaSuccess) return LOCKS_ERR_CUDA;
  ctx->prof_cap = max_steps;
  ctx->prof_n = 0;
  return LOCKS_OK;
}

int locks_profile_read(locks_ctx *ctx, float *stage_ms, locks_stream stream) {
  if (!ctx || !ctx->prof_ev || !stage_ms) return LOCKS_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LOCKS_ERR_CUDA;
  for (int s = 0; s < LOCKS_PROF_MARKS - 1; ++s)
    if (cudaEventElapsedTime(&stage_ms[s], ctx->prof_ev[s], ctx->prof_ev[s + 1]) != cudaSuccess) return LOCKS_ERR_CUDA;
  return LOCKS_OK;
}

int locks_profile_end(locks_ctx *ctx, float *stage_ms, int *steps) {
  if (!ctx || !ctx->prof_ev || !stage_ms || !steps) return LOCKS_ERR_INVALID_ARG;
  int rc = LOCKS_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) rc = LOCKS_ERR_CUDA;
  for (int s = 0; s < LOCKS_PROF_MARKS - 1; ++s) stage_ms[s] = 0.f;
  for (int i = 0; i < ctx->prof_n && rc == LOCKS_OK; ++i)
    for (int s = 0; s < LOCKS_PROF_MARKS - 1; ++s) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, ctx->prof_ev[i * LOCKS_PROF_MARKS + s], ctx->prof_ev[i * LOCKS_PROF_MARKS + s + 1]) !=
          cudaSuccess) { rc = LOCKS_ERR_CUDA; break; }
      stage_ms[s] += ms;
    }
  *steps = ctx->prof_n;
  if (ctx->prof_n > 0) for (int s = 0; s < LOCKS_PROF_MARKS - 1; ++s) stage_ms[s] /= ctx->prof_n;
  for (int i = 0; i < ctx->prof_cap * LOCKS_PROF_MARKS; ++i) cudaEventDestroy(ctx->prof_ev[i]);
  delete[] ctx->prof_ev;
  ctx->prof_ev = nullptr; ctx->prof_cap = ctx->prof_n = 0;
  return rc;
}

const char *locks_strerror(int code) {
  switch (code) {
    case LOCKS_OK: return "ok";
    case LOCKS_ERR_INVALID_ARG: return "invalid argument";
    case LOCKS_ERR_UNSUPPORTED: return "configuration not supported by the kernels";
    case LOCKS_ERR_WORKSPACE: return "workspace too small or misaligned";
    case LOCKS_ERR_CUDA: return "CUDA runtime error";
    case LOCKS_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case LOCKS_ERR_BAD_BLOCK: return "page or block id outside the cache";
    case LOCKS_ERR_TOO_LARGE: return "problem larger than the library's built-in scratch (batch * q heads too large)";
    default: return "unknown error";
  }
}

}  // extern "C"
