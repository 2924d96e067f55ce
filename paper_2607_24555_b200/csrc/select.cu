// Stage A, part 2: share-average combine and budgeted page selection (Sec. 4 of the paper):
//   log Z_g   = log sum_{j in 1..P-2} exp s^_j(q_g)                       (candidates only)
//   log m_bar_j = log( (1/G) sum_g exp(s^_j(q_g) - log Z_g) )
//   S = {0, P-1}  U  top-(k-2) candidates by log m_bar_j (ties: lower page index), ids ascending.
// Stage 1 (one 512-thread CTA per chunk of 2048 / 4096 / 8192 pages of a (request, KV head)) ranks its
// chunk with an exact 4-pass radix select over keys held in registers and compacts the winners in
// page order.  With one chunk it writes the final table; with several, log Z comes from a small
// reduction kernel, each chunk emits its own top-(k-2) (value, page) list and stage 2 re-selects
// among them (a chunk's local top-(k-2) always contains the chunk's share of the global top-(k-2),
// ties included, because both use the same lower-index tie rule and lists stay in page order).
// Pages are dealt to threads round-robin (element i of thread t is page i*512 + t), so loads are
// coalesced and every thread is busy whatever the context length.
#include "locks_internal.cuh"

namespace {

constexpr int kNW = LOCKS_SEL_THREADS / 32;

struct SelParams {
  const float *shat;
  const float2 *part;
  const int32_t *seq_lens;
  int32_t *ids, *cnt;
  float *logshare;
  float *cand_val;
  int32_t *cand_idx;
  float *logz;      // [batch][Hq] log Z_g, written by logz_kernel when a problem spans several chunks
  int32_t *status;
  int batch, Hq, Hkv, G, Pmax, max_groups, k, chunks, kc, chunk_pages, part_slots;
  locks_append app;  // decode step only: the new token's K/V rows, written here beside the ranking
};

// Decode step: the CTA of (request b, KV head h) writes the new token's K and V rows of that head into the
// cache (one warp, a few independent loads and stores beside the ranking's own loads), and the CTA of
// head 0 stores the step's length back to the caller's array.  Nothing reads the caller's array between
// the scan (complete before this kernel passes its wait) and the end of the step: the step's other
// kernels take lengths from the published copy.
__device__ __forceinline__ void append_token(const locks_append &a, int batch, int Hkv, int Pmax, int b, int h,
                                             int lane, int T, int32_t *status) {
  if (h == 0 && lane == 0) a.seq_commit[b] = T;
  const int at = a.seq_eff[batch + b];
  if (at < 0) return;
  const int page = at / LOCKS_B, slot = at % LOCKS_B;
  const int block = a.block_table[(int64_t)b * Pmax + page];
  if (block < 0 || block >= a.num_blocks) {
    if (lane == 0) set_status(status, LOCKS_ERR_BAD_BLOCK);
    return;
  }
  const int64_t dst = (int64_t)block * a.sb + (int64_t)h * a.sh + (int64_t)slot * a.st;
  const int64_t src = ((int64_t)b * Hkv + h) * LOCKS_D;
  if (a.esz == 2) {
    const uint2 kk = reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(a.k_new) + src)[lane];
    const uint2 vv = reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(a.v_new) + src)[lane];
    reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(a.k) + dst)[lane] = kk;
    reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(a.v) + dst)[lane] = vv;
  } else {
    const uint4 kk = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint32_t *>(a.k_new) + src)[lane];
    const uint4 vv = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint32_t *>(a.v_new) + src)[lane];
    reinterpret_cast<uint4 *>(reinterpret_cast<uint32_t *>(a.k) + dst)[lane] = kk;
    reinterpret_cast<uint4 *>(reinterpret_cast<uint32_t *>(a.v) + dst)[lane] = vv;
  }
}

struct SelShared {
  int hist[kNW * 256];   // one 256-bin histogram per warp
  int misc[16];          // per-pass result (double-buffered)
  int wsum[8];
  int cnt[16 * kNW];     // per (slab, warp) winner counts for the ordered compaction
  float logz[16];
};

__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exact top-K among the block's N = 512*EPT keys; element i of thread t has index i*512 + t.
// sel[i] is set for the K winners: every key above the K-th largest, plus the lowest-indexed keys
// equal to it.  pos[i] = rank of a winner in index order.  Requires K <= number of valid keys.
// Four 8-bit radix passes.  Every warp counts into its own histogram (page masses share their
// leading bits, so a shared histogram would serialise all warps on one or two counters); bin b of
// the block is then summed and suffix-scanned by thread 255 - b.  sh.hist must be zero on entry.
template <int EPT>
__device__ void block_topk(const uint32_t (&key)[EPT], int K, bool (&sel)[EPT], int (&pos)[EPT], SelShared &sh,
                           int nslab = EPT) {   // slabs >= nslab hold no valid key (uniform across the block)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (K <= 0) {  // nothing to pick (k = 2): uniform across the block
#pragma unroll
    for (int i = 0; i < EPT; ++i) { sel[i] = false; pos[i] = 0; }
    return;
  }
  uint32_t prefix = 0, mask = 0;
  int remaining = K;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    int *mine = sh.hist + warp * 256;
#pragma unroll
    for (int i = 0; i < EPT; ++i)
      if (i < nslab && (key[i] & mask) == prefix) atomicAdd(&mine[(key[i] >> shift) & 255], 1);
    __syncthreads();
    int c = 0, incl = 0;
    if (tid < 256) {   // thread t owns bin 255 - t: bins are scanned from the largest digit down
      const int bin = 255 - tid;
#pragma unroll
      for (int w = 0; w < kNW; ++w) { c += sh.hist[w * 256 + bin]; sh.hist[w * 256 + bin] = 0; }
      incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) sh.wsum[warp] = incl;
    }
    __syncthreads();
    if (tid < 256) {
      int before = incl - c;
      for (int w = 0; w < warp; ++w) before += sh.wsum[w];
      if (before < remaining && remaining <= before + c) {
        sh.misc[(pass & 1) * 2] = 255 - tid;
        sh.misc[(pass & 1) * 2 + 1] = remaining - before;
      }
    }
    __syncthreads();
    prefix |= (uint32_t)sh.misc[(pass & 1) * 2] << shift;
    mask |= 255u << shift;
    remaining = sh.misc[(pass & 1) * 2 + 1];
  }
  // prefix is the K-th largest key; `remaining` of the keys equal to it are taken, lowest index first.
  // Ordered compaction: slab i holds indices i*512 .. i*512+511, one per thread.
  uint32_t bg[EPT], be[EPT];
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    bg[i] = be[i] = 0u;
    if (i < nslab) {
      bg[i] = __ballot_sync(0xffffffffu, key[i] > prefix);
      be[i] = __ballot_sync(0xffffffffu, key[i] == prefix);
    }
    if (lane == 0) sh.cnt[i * kNW + warp] = (__popc(bg[i]) << 16) | __popc(be[i]);
  }
  __syncthreads();
  if (warp == 0) {   // exclusive scan of the EPT*kNW counts in (slab, warp) order
    constexpr int N = EPT * kNW, PER = (N + 31) / 32;
    int v[PER], tot = 0;
#pragma unroll
    for (int u = 0; u < PER; ++u) { const int e = lane * PER + u; v[u] = e < N ? sh.cnt[e] : 0; tot += v[u]; }
    int incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int x = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += x;
    }
    int run = incl - tot;
#pragma unroll
    for (int u = 0; u < PER; ++u) { const int e = lane * PER + u; if (e < N) sh.cnt[e] = run; run += v[u]; }
  }
  __syncthreads();
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    const int base = sh.cnt[i * kNW + warp];
    const int gt_before = (base >> 16) + __popc(bg[i] & lt), eq_before = (base & 0xffff) + __popc(be[i] & lt);
    const bool gt = key[i] > prefix, eq = key[i] == prefix;
    sel[i] = gt || (eq && eq_before < remaining);
    pos[i] = gt_before + min(eq_before, remaining);
  }
}

__device__ __forceinline__ void lse_merge(float &m, float &s, float om, float os) {
  const float nm = fmaxf(m, om);
  if (nm > -INFINITY) {
    s = s * __expf(m - nm) + os * __expf(om - nm);
    m = nm;
  }
}

// log Z_g of every head of the group from the scan's per-group partials -> sh_logz[g]
__device__ void group_logz(const SelParams &p, int b, int h, int ngroups, float *sh_logz) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int g = warp; g < p.G; g += kNW) {
    const float2 *pp = p.part + ((int64_t)b * p.Hq + h * p.G + g) * p.max_groups;
    float m = -INFINITY, s = 0.f;
    for (int i = lane; i < ngroups; i += 32) {
      const float2 v = pp[i];
      if (v.x > -INFINITY) lse_merge(m, s, v.x, v.y);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lse_merge(m, s, __shfl_xor_sync(0xffffffffu, m, o), __shfl_xor_sync(0xffffffffu, s, o));
    if (lane == 0) sh_logz[g] = m + __logf(s);
  }
}

// log Z_g of one query head from the scan's per-group partials (used when a problem is ranked in chunks)
__global__ void __launch_bounds__(256) logz_kernel(SelParams p) {
  __shared__ float sm_m[8], sm_s[8];
  const int hq = blockIdx.x, b = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  pdl_trigger();
  pdl_wait();
  const int T = p.seq_lens[b];
  const int P = (T + LOCKS_B - 1) / LOCKS_B;
  if (P <= p.k) return;
  const int nparts = min(p.part_slots, (P - 1 + LOCKS_GROUP - 1) / LOCKS_GROUP);
  const float2 *pp = p.part + ((int64_t)b * p.Hq + hq) * p.max_groups;
  float m = -INFINITY, s = 0.f;
  for (int i0 = threadIdx.x; i0 < nparts; i0 += 256 * 4) {   // four loads in flight per thread
    float2 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = (i0 + 256 * u < nparts) ? pp[i0 + 256 * u] : make_float2(-INFINITY, 0.f);
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (v[u].x > -INFINITY) lse_merge(m, s, v[u].x, v[u].y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) lse_merge(m, s, __shfl_xor_sync(0xffffffffu, m, o), __shfl_xor_sync(0xffffffffu, s, o));
  if (lane == 0) { sm_m[warp] = m; sm_s[warp] = s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float M = -INFINITY, S = 0.f;
    for (int w = 0; w < 8; ++w) lse_merge(M, S, sm_m[w], sm_s[w]);
    p.logz[b * p.Hq + hq] = M + __logf(S);
  }
}

template <int EPT>
__global__ void __launch_bounds__(LOCKS_SEL_THREADS) select_stage1_kernel(SelParams p) {
  __shared__ SelShared sh;
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
  for (int e = tid; e < kNW * 256; e += LOCKS_SEL_THREADS) sh.hist[e] = 0;
  pdl_trigger();
  pdl_wait();   // the scan's scores and partials
  const int T = p.seq_lens[b];
  if (p.app.k_new && chunk == 0 && tid >= LOCKS_SEL_THREADS - 32)
    append_token(p.app, p.batch, p.Hkv, p.Pmax, b, h, tid & 31, T, p.status);
  const int P = (T + LOCKS_B - 1) / LOCKS_B;
  const int64_t prob = (int64_t)b * p.Hkv + h;
  int32_t *ids = p.ids + prob * p.k;
  if (P <= p.k) {  // every page is kept
    if (chunk == 0) {
      for (int j = tid; j < p.k; j += LOCKS_SEL_THREADS) ids[j] = j < P ? j : -1;
      if (tid == 0) p.cnt[prob] = P;
    }
    return;
  }
  const int c0 = chunk * p.chunk_pages;  // first page of this chunk
  if (c0 > P - 2) {  // chunk past the candidates: emit an empty list
    if (p.chunks > 1)
      for (int j = tid; j < p.kc; j += LOCKS_SEL_THREADS) {
        p.cand_val[(prob * p.chunks + chunk) * p.kc + j] = -INFINITY;
        p.cand_idx[(prob * p.chunks + chunk) * p.kc + j] = -1;
      }
    return;
  }
  // scores of the first heads are fetched before the log Z reduction so that the two latencies overlap
  constexpr int PRE = EPT <= 8 ? 4 : 2;
  const float *row0 = p.shat + ((int64_t)b * p.Hq + h * p.G) * p.Pmax;
  bool valid[EPT];
  float raw[PRE][EPT];
  // slabs of 512 pages that hold at least one candidate of this chunk (the configured maximum context
  // is usually longer than the sequence)
  const int nslab = min(EPT, (min(P - 1, c0 + p.chunk_pages) - c0 + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS);
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    const int page = c0 + i * LOCKS_SEL_THREADS + tid;
    valid[i] = i < nslab && page >= 1 && page <= P - 2;
  }
#pragma unroll
  for (int g = 0; g < PRE; ++g)
#pragma unroll
    for (int i = 0; i < EPT; ++i)
      raw[g][i] = (g < p.G && valid[i]) ? row0[(int64_t)g * p.Pmax + c0 + i * LOCKS_SEL_THREADS + tid] : 0.f;
  if (p.chunks == 1) group_logz(p, b, h, min(p.part_slots, (P - 1 + LOCKS_GROUP - 1) / LOCKS_GROUP), sh.logz);
  else if (tid < p.G) sh.logz[tid] = p.logz[b * p.Hq + h * p.G + tid];
  __syncthreads();
  // log m_bar of this thread's pages: log mean_g exp(s^_g - log Z_g)
  float val[EPT];
  uint32_t key[EPT];
  const float logG = __logf((float)p.G);
  {
    float mx[EPT], sm[EPT];
#pragma unroll
    for (int i = 0; i < EPT; ++i) { mx[i] = -INFINITY; sm[i] = 0.f; }
#pragma unroll
    for (int g = 0; g < PRE; ++g) {
      if (g < p.G) {
        const float lz = sh.logz[g];
#pragma unroll
        for (int i = 0; i < EPT; ++i)
          if (valid[i]) lse_merge(mx[i], sm[i], raw[g][i] - lz, 1.f);
      }
    }
    for (int g = PRE; g < p.G; ++g) {
      const float *row = row0 + (int64_t)g * p.Pmax + c0 + tid;
      const float lz = sh.logz[g];
      float tv[EPT];
#pragma unroll
      for (int i = 0; i < EPT; ++i) tv[i] = (i < nslab && valid[i]) ? row[i * LOCKS_SEL_THREADS] : 0.f;
#pragma unroll
      for (int i = 0; i < EPT; ++i)
        if (valid[i]) lse_merge(mx[i], sm[i], tv[i] - lz, 1.f);
    }
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
      val[i] = valid[i] ? mx[i] + __logf(sm[i]) - logG : -INFINITY;
      key[i] = valid[i] ? order_key(val[i]) : 0u;
      if (valid[i] && p.logshare) p.logshare[prob * p.Pmax + c0 + i * LOCKS_SEL_THREADS + tid] = val[i];
    }
  }
  const int cand_in_chunk = min(P - 2, c0 + p.chunk_pages - 1) - max(1, c0) + 1;
  const int K = min(p.k - 2, cand_in_chunk);
  bool sel[EPT];
  int pos[EPT];
  block_topk<EPT>(key, K, sel, pos, sh, nslab);
  if (p.chunks == 1) {
#pragma unroll
    for (int i = 0; i < EPT; ++i)
      if (sel[i]) ids[1 + pos[i]] = c0 + i * LOCKS_SEL_THREADS + tid;
    if (tid == 0) {
      ids[0] = 0;
      ids[p.k - 1] = P - 1;
      p.cnt[prob] = p.k;
    }
  } else {
    float *cv = p.cand_val + (prob * p.chunks + chunk) * p.kc;
    int32_t *ci = p.cand_idx + (prob * p.chunks + chunk) * p.kc;
#pragma unroll
    for (int i = 0; i < EPT; ++i)
      if (sel[i]) { cv[pos[i]] = val[i]; ci[pos[i]] = c0 + i * LOCKS_SEL_THREADS + tid; }
    for (int j = K + tid; j < p.kc; j += LOCKS_SEL_THREADS) { cv[j] = -INFINITY; ci[j] = -1; }
  }
}

template <int EPT>
__global__ void __launch_bounds__(LOCKS_SEL_THREADS) select_stage2_kernel(SelParams p) {
  __shared__ SelShared sh;
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  for (int e = tid; e < kNW * 256; e += LOCKS_SEL_THREADS) sh.hist[e] = 0;
  pdl_trigger();
  pdl_wait();   // stage 1's candidate lists
  __syncthreads();
  const int T = p.seq_lens[b];
  const int P = (T + LOCKS_B - 1) / LOCKS_B;
  if (P <= p.k) return;  // stage 1 already wrote the table
  const int64_t prob = (int64_t)b * p.Hkv + h;
  const int N = p.chunks * p.kc;
  const float *cv = p.cand_val + prob * N;
  const int32_t *ci = p.cand_idx + prob * N;
  uint32_t key[EPT];
  int idx[EPT];
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    const int j = i * LOCKS_SEL_THREADS + tid;   // list position = ascending page order
    const bool ok = j < N && ci[j] >= 0;
    idx[i] = ok ? ci[j] : -1;
    key[i] = ok ? order_key(cv[j]) : 0u;
  }
  bool sel[EPT];
  int pos[EPT];
  block_topk<EPT>(key, p.k - 2, sel, pos, sh);
  int32_t *ids = p.ids + prob * p.k;
#pragma unroll
  for (int i = 0; i < EPT; ++i)
    if (sel[i]) ids[1 + pos[i]] = idx[i];
  if (tid == 0) {
    ids[0] = 0;
    ids[p.k - 1] = P - 1;
    p.cnt[prob] = p.k;
  }
}

}  // namespace

int locks_launch_select(locks_ctx *c, const float *shat, const locks_kv *kv, int batch, int32_t *ids,
                        int32_t *cnt, float *logshare, const locks_append *app, cudaStream_t st) {
  SelParams p;
  if (app) p.app = *app;
  else p.app.k_new = nullptr;
  p.status = c->status;
  p.shat = shat; p.part = c->part; p.seq_lens = kv->seq_lens; p.ids = ids; p.cnt = cnt; p.logshare = logshare;
  p.cand_val = c->cand_val; p.cand_idx = c->cand_idx;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G; p.Pmax = c->Pmax;
  p.max_groups = c->max_groups; p.k = c->k; p.chunks = c->sel_chunks; p.kc = c->sel_kc;
  p.chunk_pages = c->sel_ept * LOCKS_SEL_THREADS;
  p.logz = c->logz;
  p.part_slots = c->part_slots;
  if (c->sel_chunks > 1) {
    locks_launch_pdl(logz_kernel, dim3(p.Hq, batch), dim3(256), 0, st, p);
    int rc0 = locks_check_launch(c);
    if (rc0 != LOCKS_OK) return rc0;
  }
  dim3 g1(c->sel_chunks, p.Hkv, batch);
  if (c->sel_ept == 4) locks_launch_pdl(select_stage1_kernel<4>, g1, dim3(LOCKS_SEL_THREADS), 0, st, p);
  else if (c->sel_ept == 8) locks_launch_pdl(select_stage1_kernel<8>, g1, dim3(LOCKS_SEL_THREADS), 0, st, p);
  else locks_launch_pdl(select_stage1_kernel<16>, g1, dim3(LOCKS_SEL_THREADS), 0, st, p);
  int rc = locks_check_launch(c);
  if (rc != LOCKS_OK || c->sel_chunks == 1) return rc;
  const int N = c->sel_chunks * c->sel_kc;
  const int ept = (N + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS;
  dim3 grid(p.Hkv, batch);
  if (ept <= 4) locks_launch_pdl(select_stage2_kernel<4>, grid, dim3(LOCKS_SEL_THREADS), 0, st, p);
  else if (ept <= 16) locks_launch_pdl(select_stage2_kernel<16>, grid, dim3(LOCKS_SEL_THREADS), 0, st, p);
  else return LOCKS_ERR_UNSUPPORTED;
  return locks_check_launch(c);
}
