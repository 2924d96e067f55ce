// Stage A, part 2: share-average combine and budgeted page selection (Sec. 4 of the paper):
//   log Z_g   = log sum_{j in 1..P-2} exp s^_j(q_g)                       (candidates only)
//   log m_bar_j = log( (1/G) sum_g exp(s^_j(q_g) - log Z_g) )
//   S = {0, P-1}  U  top-(k-2) candidates by log m_bar_j (ties: lower page index), ids ascending.
// One 512-thread CTA ranks a chunk of 2048 / 4096 / 8192 pages of a (request, KV head): it turns the
// chunk's scores into order-preserving 32-bit keys in shared memory, finds the (k-2)-th largest with an
// exact 4-pass radix select and compacts the winners in page order.  With one chunk per problem that is
// the final table.  With several, each chunk emits its own top-(k-2) (value, page) list, and the CTA of a
// problem that finishes last ranks the lists the same way in the same launch (a chunk's local top-(k-2)
// always contains the chunk's share of the global top-(k-2), ties included, because both rounds use the
// same lower-index tie rule and lists stay in page order).
// Pages are dealt to threads round-robin (element i of thread t is page i*512 + t), so loads are
// coalesced and every thread is busy whatever the context length.
// The kernel runs once through its code on at most a few dozen SMs, so instruction fetch is a visible part
// of its latency: loops over a thread's elements stay rolled (keys live in shared memory, not in
// registers), and the two routines used by both rounds are real calls.
#include "locks_internal.cuh"

namespace {

constexpr int kNW = LOCKS_SEL_THREADS / 32;
constexpr int kMaxKeys = LOCKS_SEL_MAX_EPT * LOCKS_SEL_THREADS;   // keys one CTA ranks at most
constexpr int kMaxWin = 4 * LOCKS_SEL_THREADS;                    // k - 2 at most (checked on the host)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct SelParams {
  const float *shat;
  const float2 *part;
  const int32_t *seq_lens;
  const int32_t *part_cnt;   // partials per head of each problem, or nullptr: part_slots for all
  int pc_div;                // rankings per entry of part_cnt (1; per-head arm: G)
  int32_t *ids, *cnt;
  float *logshare;
  uint32_t *cand_key;  // [batch][Hkv][chunks][kc] chunk lists (chunked selection only): keys, 0 = no entry
  int32_t *cand_idx;
  int32_t *sel_done;   // [batch][Hkv] chunk-arrival counters (zero between launches)
  int32_t *status;
  int batch, Hq, Hkv, G, Pmax, max_groups, k, chunks, kc, chunk_pages, part_slots;
  int combine;       // LOCKS_COMBINE_*
  int Bshift;        // log2 of the page size (4, 5 or 6)
  locks_append app;  // decode step only: the new token's K/V rows, written here beside the ranking
};

// Decode step: the CTA of (request b, KV head h) writes the new token's K and V rows of that head into the
// cache (one warp, a few independent loads and stores beside the ranking's own loads), and the CTA of
// head 0 stores the step's length back to the caller's array.  Nothing reads the caller's array between
// the scan (complete before this kernel passes its wait) and the end of the step: the step's other
// kernels take lengths from the published copy.
__device__ __forceinline__ void append_token(const locks_append &a, int batch, int Hkv, int Pmax, int b, int h,
                                             int lane, int T, int32_t *status, int Bshift) {
  if (h == 0 && lane == 0) a.seq_commit[b] = T;
  const int at = a.seq_eff[batch + b];
  if (at < 0) return;
  const int page = at >> Bshift, slot = at & ((1 << Bshift) - 1);
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
  uint32_t key[kMaxKeys];             // order-preserving keys, element i of thread t at i*512 + t
  int hist[3 * 256];                  // radix histograms, rotating
  __align__(16) int cnt[256];         // per (slab, warp) winner counts for the ordered compaction
  int misc[16];                       // per-pass result (double-buffered), arrival flag
  float lz2[16];                      // log2-domain log Z_g
  float lzm[kNW], lzs[kNW];           // per-warp (max, sum) of the log Z reduction
  uint32_t red[2 * kNW];              // per-warp AND / OR of the keys
  int win[kMaxWin];                   // final round: entry index of winner number pos
};

extern __shared__ __align__(16) uint8_t sel_smem[];
// The routines below are real calls; each takes the block's shared state from the symbol itself (a
// reference argument would turn every access into a generic one) and its inputs by value (no stack).
__device__ __forceinline__ SelShared &shared_state() { return *reinterpret_cast<SelShared *>(sel_smem); }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2f(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// K-th largest of the keys sh.key[i*512 + t], i < nslab (invalid elements hold key 0; 1 <= K <= number of
// valid keys).  Returns (key, how many of the keys equal to it belong to the top K).
// Radix passes of up to 8 bits from the top over the keys' offsets from the smallest valid key (one MIN / MAX
// reduction first).  A pass costs one barrier: all warps count into
// one 256-bin histogram, then every warp scans it on its own (lane l owns bins 8 (31 - l) .. + 7, so
// lane order is descending digit order) while the histogram of the next pass -- three rotate -- is
// already being filled by warps that are ahead.
__device__ __noinline__ uint2 radix_select(int nslab, int K) {
  SelShared &sh = shared_state();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < 256) sh.hist[tid] = 0;
  uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll 4
  for (int i = 0; i < nslab; ++i) {
    const uint32_t k = sh.key[i * LOCKS_SEL_THREADS + tid];
    if (k) { kmin = min(kmin, k); kmax = max(kmax, k); }
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { sh.red[warp] = kmin; sh.red[kNW + warp] = kmax; }
  __syncthreads();
  kmin = __reduce_min_sync(0xffffffffu, sh.red[lane & (kNW - 1)]);
  kmax = __reduce_max_sync(0xffffffffu, sh.red[kNW + (lane & (kNW - 1))]);
  // The passes rank the keys' offsets from the smallest valid key: page masses lie within a few units of each
  // other, so the offsets need far fewer than 32 bits (typically 24: three passes), and the first pass already
  // works on bits in which the keys differ, which spreads them over the bins (hundreds of atomics on two or
  // three counters would serialise); the later passes see only the few keys of the threshold bin.
  const int bits = 32 - __clz(kmax - kmin);   // 0: all valid keys are equal (kmax >= kmin: K >= 1 valid keys)
  uint32_t mask = 0u, prefix = 0u;            // decided leading bits of the offset of the K-th largest key
  int remaining = K;
  int cur = 0;
#pragma unroll 1
  for (int left = bits; left > 0;) {   // bits not yet decided
    const int width = min(8, left), shift = left - width;
    const uint32_t dmask = (1u << width) - 1u;
    left = shift;
    const int nxt = cur == 2 ? 0 : cur + 1;
    int *hc = sh.hist + cur * 256;
    if (tid < 256) sh.hist[nxt * 256 + tid] = 0;   // last read two passes ago
#pragma unroll 4
    for (int i = 0; i < nslab; ++i) {
      const uint32_t k = sh.key[i * LOCKS_SEL_THREADS + tid], d = k - kmin;
      if (k && (d & mask) == prefix) atomicAdd(&hc[(d >> shift) & dmask], 1);
    }
    __syncthreads();
    const int base = 8 * (31 - lane);
    const int4 lo = *reinterpret_cast<const int4 *>(hc + base), hi = *reinterpret_cast<const int4 *>(hc + base + 4);
    const int c[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    const int tot = (c[0] + c[1]) + (c[2] + c[3]) + (c[4] + c[5]) + (c[6] + c[7]);
    int incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    const bool hit = incl - tot < remaining && remaining <= incl;   // the K-th largest falls in this lane's bins
    int digit = 0, rem = 0, acc = incl - tot;
#pragma unroll
    for (int j = 7; j >= 0; --j) {
      if (hit && acc < remaining && remaining <= acc + c[j]) { digit = base + j; rem = remaining - acc; }
      acc += c[j];
    }
    const uint32_t who = __ballot_sync(0xffffffffu, hit);
    const int src = who ? __ffs(who) - 1 : 0;
    digit = __shfl_sync(0xffffffffu, digit, src);
    remaining = __shfl_sync(0xffffffffu, rem, src);
    prefix |= (uint32_t)digit << shift;
    mask |= dmask << shift;
    cur = nxt;
  }
  return make_uint2(kmin + prefix, (uint32_t)remaining);
}

enum { kEmitIds = 0, kEmitList = 1, kEmitFinal = 2 };

// Winners = keys above `prefix` plus the first `remaining` keys equal to it, in element order.  Winner
// number `pos` (< cap) of element e is written as
//   kEmitIds:   ids[1 + pos] = c0 + e                         (final table of a single-chunk problem)
//   kEmitList:  list_key[pos] = key, list_idx[pos] = c0 + e   (a chunk's candidate list)
//   kEmitFinal: ids[1 + pos] = list_idx[e]                    (final table from the problem's lists)
__device__ __noinline__ void compact_emit(int nslab, uint32_t prefix, int remaining, int cap, int mode,
                                          int c0, int32_t *ids, uint32_t *list_key, int32_t *list_idx) {
  SelShared &sh = shared_state();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (mode == kEmitFinal)
    for (int j = tid; j < cap; j += LOCKS_SEL_THREADS) sh.win[j] = 0;   // a slot no winner fills still names a real entry
  __syncthreads();   // the previous user of sh.cnt is done
#pragma unroll 2
  for (int i = 0; i < nslab; ++i) {
    const uint32_t k = sh.key[i * LOCKS_SEL_THREADS + tid];
    const uint32_t bg = __ballot_sync(0xffffffffu, k > prefix), be = __ballot_sync(0xffffffffu, k == prefix);
    if (lane == 0) sh.cnt[i * kNW + warp] = (__popc(bg) << 16) | __popc(be);
  }
  __syncthreads();
  if (warp == 0) {   // exclusive scan of the nslab * kNW (<= 256) counts in (slab, warp) order, 8 per lane
    const int n = nslab * kNW;
    int4 *q = reinterpret_cast<int4 *>(sh.cnt + lane * 8);
    int4 lo = q[0], hi = q[1];
    int c[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    int tot = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) { if (lane * 8 + j >= n) c[j] = 0; tot += c[j]; }
    int incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    int run = incl - tot;
#pragma unroll
    for (int j = 0; j < 8; ++j) { const int v = c[j]; c[j] = run; run += v; }
    q[0] = make_int4(c[0], c[1], c[2], c[3]);
    q[1] = make_int4(c[4], c[5], c[6], c[7]);
  }
  __syncthreads();
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll 2
  for (int i = 0; i < nslab; ++i) {
    const int e = i * LOCKS_SEL_THREADS + tid;
    const uint32_t k = sh.key[e];
    const bool gt = k > prefix, eq = k == prefix;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const int base = sh.cnt[i * kNW + warp];
    const int gt_before = (base >> 16) + __popc(bg & lt), eq_before = (base & 0xffff) + __popc(be & lt);
    const int pos = gt_before + min(eq_before, remaining);
    if ((gt || (eq && eq_before < remaining)) && pos < cap) {
      if (mode == kEmitIds) ids[1 + pos] = c0 + e;
      else if (mode == kEmitList) { list_key[pos] = k; list_idx[pos] = c0 + e; }
      else sh.win[pos] = e;   // the page of entry e is fetched below, all winners at once
    }
  }
  if (mode == kEmitFinal) {
    __syncthreads();
    for (int j0 = tid; j0 < cap; j0 += 4 * LOCKS_SEL_THREADS) {
      int v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { const int j = j0 + u * LOCKS_SEL_THREADS; v[u] = j < cap ? __ldcg(list_idx + sh.win[j]) : 0; }
#pragma unroll
      for (int u = 0; u < 4; ++u) { const int j = j0 + u * LOCKS_SEL_THREADS; if (j < cap) ids[1 + j] = v[u]; }
    }
  }
}

// log Z_g of every head of the group from the scan's partials (max_i, sum_i), part0 = head 0's row,
// -> sh.lz2[g] (log2 domain):
// log2 Z = M + log2 sum_i sum_i 2^(max_i - M), M = max_i max_i.  The block's warps are dealt to (head, slice)
// pairs; a lane keeps eight loads in flight.  Ends with the block synchronised.
__device__ __noinline__ void group_logz(const float2 *part0, int G, int max_groups, int nparts) {
  SelShared &sh = shared_state();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gw = min(G, kNW);            // heads handled per round
  const int nslice = max(1, kNW / G);    // warps per head
#pragma unroll 1
  for (int g0 = 0; g0 < G; g0 += kNW) {  // one round unless G > 16
    const int slice = warp / gw, g = g0 + warp - slice * gw;
    float m = -INFINITY, s = 0.f;
    if (g < G && slice < nslice) {
      const float2 *pp = part0 + (int64_t)g * max_groups;
#pragma unroll 1
      for (int i0 = slice * 32 + lane; i0 < nparts; i0 += 256 * nslice) {
        float2 v[8];   // eight loads in flight: up to 256 partials of a head in one round trip
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (i0 + 32 * nslice * u < nparts) ? pp[i0 + 32 * nslice * u] : make_float2(-INFINITY, 0.f);
        float nm = m;
#pragma unroll
        for (int u = 0; u < 8; ++u) nm = fmaxf(nm, v[u].x);
        if (nm > -INFINITY) {
          s *= ex2f((m - nm) * kLog2e);
#pragma unroll
          for (int u = 0; u < 8; ++u) s = fmaf(v[u].y, ex2f((v[u].x - nm) * kLog2e), s);
          m = nm;
        }
      }
      float M = m;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      s = M > -INFINITY ? s * ex2f((m - M) * kLog2e) : 0.f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      m = M;
    }
    if (lane == 0) { sh.lzm[warp] = m; sh.lzs[warp] = s; }
    __syncthreads();
    if (threadIdx.x < min(G - g0, kNW)) {
      float M = -INFINITY, S = 0.f;
#pragma unroll 1
      for (int sl = 0; sl < nslice; ++sl) M = fmaxf(M, sh.lzm[sl * gw + threadIdx.x]);
#pragma unroll 1
      for (int sl = 0; sl < nslice; ++sl) {
        const float wm = sh.lzm[sl * gw + threadIdx.x];
        if (wm > -INFINITY) S = fmaf(sh.lzs[sl * gw + threadIdx.x], ex2f((wm - M) * kLog2e), S);
      }
      sh.lz2[g0 + threadIdx.x] = M * kLog2e + lg2f(S);
    }
    __syncthreads();
  }
}

// Keys of a chunk: log m_bar of page c0 + i*512 + t as an order-preserving integer in sh.key[i*512 + t]
// (0 for pages that are not candidates).  Scores are fetched in batches of (16 / SB) heads x SB slabs, 16
// loads in flight per thread, the next batch while the current one is reduced; the first batch is in
// flight during the log Z reduction.  Per page a running (max, sum) over the heads, log2 domain.
// combine: share-average (the paper's rule) subtracts log Z_g per head and averages; group-mass sums the raw
// masses (log Z_g = 0, no 1/G); group-max keeps the largest raw score.
template <int SB>
__device__ __noinline__ void chunk_keys(const float *shat0, const float2 *part0, float *logshare0, int G, int Pmax,
                                        int max_groups, int nparts, int c0, int nslab, int P, int combine) {
  constexpr int HB = 16 / SB;
  SelShared &sh = shared_state();
  const int tid = threadIdx.x;
  const float *row0 = shat0 + c0 + tid;   // shat0: scores of the group's head 0, page 0
  const int nG = (G + HB - 1) / HB, nb = ((nslab + SB - 1) / SB) * nG;
  float cur[HB][SB], nxt[HB][SB];
  auto load = [&](int i0, int g0, float (&x)[HB][SB]) {
    bool ok[SB];
#pragma unroll
    for (int sl = 0; sl < SB; ++sl) {
      const int page = c0 + (i0 + sl) * LOCKS_SEL_THREADS + tid;
      ok[sl] = i0 + sl < nslab && page >= 1 && page <= P - 2;
    }
    const float *r = row0 + g0 * Pmax + i0 * LOCKS_SEL_THREADS;   // offsets within one request fit 32 bits
#pragma unroll
    for (int u = 0; u < HB; ++u)
#pragma unroll
      for (int sl = 0; sl < SB; ++sl)
        x[u][sl] = (ok[sl] && g0 + u < G) ? r[u * Pmax + sl * LOCKS_SEL_THREADS] : -INFINITY;
  };
  load(0, 0, cur);
  if (combine == LOCKS_COMBINE_SHARE_AVG) {
    group_logz(part0, G, max_groups, nparts);
  } else {
    if (tid < 16) sh.lz2[tid] = 0.f;
    __syncthreads();
  }
  const float logG = combine == LOCKS_COMBINE_SHARE_AVG ? __logf((float)G) : 0.f;
  float m[SB], s[SB];
#pragma unroll
  for (int sl = 0; sl < SB; ++sl) { m[sl] = -INFINITY; s[sl] = 0.f; }
  int i0 = 0, g0 = 0;
#pragma unroll 1
  for (int bi = 0; bi < nb; ++bi) {
    int i1 = i0, g1 = g0 + HB;   // the batch after this one
    if (g1 >= G) { g1 = 0; i1 += SB; }
    if (bi + 1 < nb) load(i1, g1, nxt);
#pragma unroll
    for (int sl = 0; sl < SB; ++sl) {
      float bm = -INFINITY;
#pragma unroll
      for (int u = 0; u < HB; ++u) {
        cur[u][sl] = fmaf(cur[u][sl], kLog2e, g0 + u < G ? -sh.lz2[g0 + u] : 0.f);   // heads past the group stay -inf
        bm = fmaxf(bm, cur[u][sl]);
      }
      const float nm = fmaxf(m[sl], bm);
      float acc = s[sl] * ex2f(m[sl] - nm);
#pragma unroll
      for (int u = 0; u < HB; ++u) acc += ex2f(cur[u][sl] - nm);
      s[sl] = acc;
      m[sl] = nm;
    }
    if (g0 + HB >= G) {   // all heads seen: keys of these slabs
#pragma unroll
      for (int sl = 0; sl < SB; ++sl) {
        const int i = i0 + sl, page = c0 + i * LOCKS_SEL_THREADS + tid;
        if (i < nslab) {
          const bool valid = page >= 1 && page <= P - 2;
          const float val = (combine == LOCKS_COMBINE_GROUP_MAX ? m[sl] : m[sl] + lg2f(s[sl])) * kLn2 - logG;
          sh.key[i * LOCKS_SEL_THREADS + tid] = valid ? order_key(val) : 0u;
          if (valid && logshare0) logshare0[page] = val;
        }
        m[sl] = -INFINITY;
        s[sl] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < HB; ++u)
#pragma unroll
      for (int sl = 0; sl < SB; ++sl) cur[u][sl] = nxt[u][sl];
    i0 = i1;
    g0 = g1;
  }
}

// Several chunks per problem: the chunk that arrives last ranks the problem's candidate lists.
__device__ __noinline__ void select_finish(int32_t *done, int chunks, int kc, int k, int32_t *ids, int32_t *count,
                                           const uint32_t *ck, const int32_t *ci, int P) {
  SelShared &sh = shared_state();
  const int tid = threadIdx.x;
  __threadfence();   // this chunk's list before its arrival
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(done, 1);
    const bool last = ticket == chunks - 1;
    if (last) *done = 0;   // every chunk has arrived: ready for the next launch
    sh.misc[8] = last;
  }
  __syncthreads();
  if (!sh.misc[8]) return;
  __threadfence();
  const int K2 = k - 2;
  // entries in list order (chunk, position) = page order; element i of thread t is entry i*512 + t
  const int N = chunks * kc;
  const int nslab = (N + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS;
#pragma unroll 4
  for (int i = 0; i < nslab; ++i) {
    const int e = i * LOCKS_SEL_THREADS + tid;
    sh.key[e] = e < N ? __ldcg(ck + e) : 0u;
  }
  if (K2 > 0) {
    const uint2 r = radix_select(nslab, K2);
    compact_emit(nslab, r.x, (int)r.y, K2, kEmitFinal, 0, ids, nullptr, const_cast<int32_t *>(ci));
  }
  if (tid == 0) {
    ids[0] = 0;
    ids[k - 1] = P - 1;
    *count = k;
  }
}

__global__ void __launch_bounds__(LOCKS_SEL_THREADS, 2) select_kernel(SelParams p) {
  SelShared &sh = shared_state();
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
  pdl_trigger();
  pdl_wait();   // the scan's scores and partials
  const int T = p.seq_lens[b];
  if (p.app.k_new && chunk == 0 && tid >= LOCKS_SEL_THREADS - 32)
    append_token(p.app, p.batch, p.Hkv, p.Pmax, b, h, tid & 31, T, p.status, p.Bshift);
  const int P = (T + (1 << p.Bshift) - 1) >> p.Bshift;
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
  if (c0 > P - 2) {  // chunk past the candidates: an empty list
    if (p.chunks > 1) {
      for (int j = tid; j < p.kc; j += LOCKS_SEL_THREADS) p.cand_key[(prob * p.chunks + chunk) * p.kc + j] = 0u;
      select_finish(p.sel_done + prob, p.chunks, p.kc, p.k, ids, p.cnt + prob, p.cand_key + prob * p.chunks * p.kc,
                    p.cand_idx + prob * p.chunks * p.kc, P);
    }
    return;
  }
  // slabs of 512 pages that hold at least one candidate of this chunk (the configured maximum context
  // is usually longer than the sequence)
  const int nslab = (min(P - 1, c0 + p.chunk_pages) - c0 + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS;
  {
    const float *shat0 = p.shat + ((int64_t)b * p.Hq + h * p.G) * p.Pmax;
    const float2 *part0 = p.part + ((int64_t)b * p.Hq + h * p.G) * p.max_groups;
    float *ls0 = p.logshare ? p.logshare + prob * p.Pmax : nullptr;
    const int nparts = p.part_cnt ? min(max(p.part_cnt[prob / p.pc_div], 0), p.max_groups)
                                  : min(p.part_slots, (P - 1 + LOCKS_GROUP - 1) / LOCKS_GROUP);
    if (nslab >= 3) chunk_keys<4>(shat0, part0, ls0, p.G, p.Pmax, p.max_groups, nparts, c0, nslab, P, p.combine);
    else if (nslab == 2) chunk_keys<2>(shat0, part0, ls0, p.G, p.Pmax, p.max_groups, nparts, c0, nslab, P, p.combine);
    else chunk_keys<1>(shat0, part0, ls0, p.G, p.Pmax, p.max_groups, nparts, c0, nslab, P, p.combine);
  }
  const int cand_in_chunk = min(P - 2, c0 + p.chunk_pages - 1) - max(1, c0) + 1;
  const int K = min(p.k - 2, cand_in_chunk);
  uint2 kth = make_uint2(0xFFFFFFFFu, 0u);
  if (K > 0) kth = radix_select(nslab, K);
  if (p.chunks == 1) {
    if (K > 0) compact_emit(nslab, kth.x, (int)kth.y, K, kEmitIds, c0, ids, nullptr, nullptr);
    if (tid == 0) {
      ids[0] = 0;
      ids[p.k - 1] = P - 1;
      p.cnt[prob] = p.k;
    }
  } else {
    uint32_t *lk = p.cand_key + (prob * p.chunks + chunk) * p.kc;
    for (int j = K + tid; j < p.kc; j += LOCKS_SEL_THREADS) lk[j] = 0u;   // fewer candidates than list slots
    if (K > 0) compact_emit(nslab, kth.x, (int)kth.y, K, kEmitList, c0, nullptr, lk, p.cand_idx + (prob * p.chunks + chunk) * p.kc);
    select_finish(p.sel_done + prob, p.chunks, p.kc, p.k, ids, p.cnt + prob, p.cand_key + prob * p.chunks * p.kc,
                  p.cand_idx + prob * p.chunks * p.kc, P);
  }
}

// ---- page-sharded selection (one long request whose pages are dealt to several GPUs) -----------------------
// log Z_g of the pages one shard scanned, from the scan's partials: one warp per (request, query head)
__global__ void __launch_bounds__(32) head_logz_kernel(const float2 *part, const int32_t *part_cnt, const int32_t *seq_lens,
                                                       float *logz, int Hq, int Hkv, int max_groups, int part_slots, int k) {
  const int hq = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
  pdl_wait();
  const int P = (seq_lens[b] + LOCKS_B - 1) / LOCKS_B;
  const int64_t prob = (int64_t)b * Hkv + hq / (Hq / Hkv);
  int nparts = part_cnt ? min(max(part_cnt[prob], 0), max_groups) : min(part_slots, (P - 1 + LOCKS_GROUP - 1) / LOCKS_GROUP);
  if (P <= k) nparts = 0;
  const float2 *pp = part + ((int64_t)b * Hq + hq) * max_groups;
  float m = -INFINITY, s = 0.f;
  for (int i = lane; i < nparts; i += 32) {
    const float2 x = pp[i];
    const float nm = fmaxf(m, x.x);
    if (nm > -INFINITY) { s = s * __expf(m - nm) + x.y * __expf(x.x - nm); m = nm; }
  }
  const float M = warp_max(m);
  s = warp_sum(M > -INFINITY ? s * __expf(m - M) : 0.f);
  if (lane == 0) logz[(int64_t)b * Hq + hq] = M > -INFINITY ? M + __logf(s) : -INFINITY;
}

// the shards' log Z values as the selector's partials: slot r of head g holds (log Z_g of shard r, 1)
__global__ void __launch_bounds__(128) ext_partials_kernel(const float *logz_parts, int nparts, float2 *part, int32_t *part_cnt,
                                                           int batch, int Hq, int Hkv, int max_groups) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < batch * Hkv) part_cnt[i] = nparts;
  if (i >= batch * Hq) return;
  for (int r = 0; r < nparts; ++r) {
    const float v = logz_parts[(int64_t)r * batch * Hq + i];
    part[(int64_t)i * max_groups + r] = make_float2(v, v > -INFINITY ? 1.f : 0.f);
  }
}

// Global top-(k-2) of the shards' candidate lists (each in page order, shards in page order, so that list order
// is page order and the lower-page tie rule carries over): one CTA per (request, KV head).
__global__ void __launch_bounds__(LOCKS_SEL_THREADS) merge_selection_kernel(const float *cand_key, const int32_t *cand_page, int nparts,
                                                                           int batch, int Hkv, int kc, int32_t *ids, int32_t *cnt) {
  SelShared &sh = shared_state();
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int64_t prob = (int64_t)b * Hkv + h, nprob = (int64_t)batch * Hkv;
  const int N = nparts * kc, nslab = (N + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS;
  int32_t *out = ids + prob * kc;
  __shared__ int s_valid;
  if (tid == 0) s_valid = 0;
  __syncthreads();
  int mine = 0;
  for (int i = 0; i < nslab; ++i) {
    const int e = i * LOCKS_SEL_THREADS + tid;
    uint32_t key = 0u;
    if (e < N) {
      const int r = e / kc, j = e - r * kc;
      const int64_t at = ((int64_t)r * nprob + prob) * kc + j;
      if (cand_page[at] >= 0) { key = order_key(cand_key[at]); ++mine; }
    }
    sh.key[e] = key;
  }
  for (int j = tid; j < kc; j += LOCKS_SEL_THREADS) out[j] = -1;
  if (mine) atomicAdd(&s_valid, mine);
  __syncthreads();
  const int K = min(kc, s_valid);
  if (K > 0) {
    const uint2 r = radix_select(nslab, K);
    compact_emit(nslab, r.x, (int)r.y, K, kEmitIds, 0, out - 1, nullptr, nullptr);   // out[pos] = winning entry, in list order
    __syncthreads();
    int page[(kMaxWin + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS];
#pragma unroll
    for (int u = 0; u < (kMaxWin + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS; ++u) {
      const int j = tid + u * LOCKS_SEL_THREADS;
      page[u] = -1;
      if (j < K) {
        const int e = out[j], rr = e / kc, jj = e - rr * kc;
        page[u] = cand_page[((int64_t)rr * nprob + prob) * kc + jj];
      }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < (kMaxWin + LOCKS_SEL_THREADS - 1) / LOCKS_SEL_THREADS; ++u)
      if (tid + u * LOCKS_SEL_THREADS < K) out[tid + u * LOCKS_SEL_THREADS] = page[u];
  }
  if (tid == 0) cnt[prob] = K;
}

}  // namespace

int locks_launch_head_logz(locks_ctx *c, const locks_kv *kv, int batch, float *logz, cudaStream_t st) {
  locks_launch_pdl(head_logz_kernel, dim3(c->cfg.num_q_heads, batch), dim3(32), 0, st, (const float2 *)c->part,
                   (const int32_t *)(c->part_balanced ? c->part_cnt : nullptr), (const int32_t *)kv->seq_lens, logz,
                   c->cfg.num_q_heads, c->cfg.num_kv_heads, c->max_groups, c->part_slots, c->k);
  return locks_check_launch(c);
}

int locks_launch_ext_partials(locks_ctx *c, const float *logz_parts, int nparts, int batch, cudaStream_t st) {
  if (nparts < 1 || nparts > c->max_groups) return LOCKS_ERR_INVALID_ARG;
  const int n = batch * c->cfg.num_q_heads;
  ext_partials_kernel<<<(n + 127) / 128, 128, 0, st>>>(logz_parts, nparts, c->part, c->part_cnt, batch, c->cfg.num_q_heads,
                                                       c->cfg.num_kv_heads, c->max_groups);
  c->part_slots = nparts;
  c->part_balanced = 1;   // the selector takes the count from part_cnt
  return locks_check_launch(c);
}

int locks_launch_merge_selection(locks_ctx *c, const float *cand_key, const int32_t *cand_page, int nparts, int batch,
                                 int32_t *ids, int32_t *cnt, cudaStream_t st) {
  if (nparts < 1 || (int64_t)nparts * c->sel_kc > kMaxKeys) return LOCKS_ERR_UNSUPPORTED;
  if (locks_attrs_needed(LOCKS_ATTR_SELECT))
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 116 * 1024);
  merge_selection_kernel<<<dim3(c->cfg.num_kv_heads, batch), LOCKS_SEL_THREADS, sizeof(SelShared), st>>>(
      cand_key, cand_page, nparts, batch, c->cfg.num_kv_heads, c->sel_kc, ids, cnt);
  return locks_check_launch(c);
}

int locks_launch_select(locks_ctx *c, const float *shat, const locks_kv *kv, int batch, int32_t *ids,
                        int32_t *cnt, float *logshare, const locks_append *app, cudaStream_t st) {
  SelParams p;
  if (app) p.app = *app;
  else p.app.k_new = nullptr;
  p.status = c->status;
  p.shat = shat; p.part = c->part; p.seq_lens = kv->seq_lens; p.ids = ids; p.cnt = cnt; p.logshare = logshare;
  p.cand_key = reinterpret_cast<uint32_t *>(c->cand_val); p.cand_idx = c->cand_idx; p.sel_done = c->sel_done;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G; p.Pmax = c->Pmax;
  p.max_groups = c->max_groups; p.k = c->k; p.chunks = c->sel_chunks; p.kc = c->sel_kc;
  p.chunk_pages = c->sel_ept * LOCKS_SEL_THREADS;
  p.part_slots = c->part_slots;
  p.combine = c->cfg.combine;
  p.pc_div = 1;
  if (p.combine == LOCKS_COMBINE_PER_HEAD) {   // every query head is a group of one with a page table of its own
    if (app) return LOCKS_ERR_UNSUPPORTED;
    p.pc_div = p.G; p.Hkv = p.Hq; p.G = 1; p.combine = LOCKS_COMBINE_SHARE_AVG;
  }
  p.Bshift = c->B == 64 ? 6 : (c->B == 32 ? 5 : 4);
  p.part_cnt = c->part_balanced ? c->part_cnt : nullptr;
  if (p.chunk_pages > kMaxKeys || (int64_t)c->sel_chunks * c->sel_kc > kMaxKeys || p.G > 16) return LOCKS_ERR_UNSUPPORTED;
  // Two CTAs fit on an SM (64 registers per thread).  That halves the waves of a launch with many more CTAs
  // than SMs, but with up to about 1.5 CTAs per SM the block scheduler stacks pairs on the SMs that drain first
  // while others idle (measured: +15 us at 192 CTAs); such launches ask for enough shared memory to keep one
  // CTA per SM.
  constexpr int kSmemAlone = 116 * 1024;
  if (locks_attrs_needed(LOCKS_ATTR_SELECT))
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemAlone);
  const int64_t nctas = (int64_t)c->sel_chunks * p.Hkv * batch;
  const size_t smem = 2 * nctas <= 3 * (int64_t)c->num_sms ? (size_t)kSmemAlone : sizeof(SelShared);
  locks_launch_pdl(select_kernel, dim3(c->sel_chunks, p.Hkv, batch), dim3(LOCKS_SEL_THREADS), smem, st, p);
  return locks_check_launch(c);
}
