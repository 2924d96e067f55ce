// Stage B: sparse paged attention over the selected pages (Sec. 3 "Decode-time attention", App. E):
//   o_g = sum_i softmax_i(q_g . k_i / sqrt(d)) v_i   over tokens i < T of the pages in the table,
// computed split-K: every CTA takes a slice of the page list, every warp streams whole pages
// (K tile 16x128 + V tile 16x128) through its own two-stage shared-memory ring with 16-byte async
// copies into an XOR-swizzled layout, scores them with m16n8k16 bf16 MMAs (the G query heads of the
// KV head are the M rows), keeps a running (max, sum, O) per head, and the CTA merges its warps by
// log-sum-exp.  Partial (o, lse) per split are merged by a second small kernel.
// A NULL page table means "all pages": the same kernel is the dense flash-decode baseline.
#include <cooperative_groups.h>
#include <mutex>
#include "locks_internal.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct AttParams {
  const void *q;
  const void *k, *v;
  int64_t sb, sh, st;
  const int32_t *block_table;
  const int32_t *seq_lens;
  const int32_t *ids, *cnt;
  float *part_o, *part_lse;
  void *out;
  float *lse;
  int32_t *status;
  int32_t *done;   // [batch*Hkv] split-arrival counters (zero between launches)
  int batch, Hq, Hkv, G, Pmax, kbud, num_blocks, splits, pages_per_cta;
  int B;             // tokens per page (the bf16 kernels: 16 only)
  int kvdiv;         // the KV head of problem h is h / kvdiv (1; per-head page tables: G, with G = 1 and Hkv = Hq here)
  int fused_merge;   // 1: the last CTA of a problem merges its splits; 0: a separate merge kernel follows
  int cluster;       // 1: the splits of a problem form one thread-block cluster and merge through its shared memory
  float sm_scale;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

constexpr int kTile = LOCKS_B * LOCKS_D * 2;                 // 4096 B: one K or V page tile in bf16
constexpr int kAttStage = 2 * kTile;                         // K + V
constexpr int kAttStages = LOCKS_ATT_STAGES;                  // ring depth per warp
constexpr int kAttSmem = LOCKS_ATT_WARPS * kAttStages * kAttStage;

// Resolve the idx-th page of this problem's list: logical page, physical block, valid tokens.
__device__ __forceinline__ bool resolve_page(const AttParams &p, int b, int64_t prob, int idx, int T, int &block,
                                             int &ntok) {
  const int page = p.ids ? p.ids[prob * p.kbud + idx] : idx;
  if (page < 0 || page >= p.Pmax) { set_status(p.status, LOCKS_ERR_BAD_BLOCK); return false; }
  block = p.block_table[(int64_t)b * p.Pmax + page];
  if (block < 0 || block >= p.num_blocks) { set_status(p.status, LOCKS_ERR_BAD_BLOCK); return false; }
  ntok = min(p.B, T - page * p.B);
  return ntok > 0;
}

__device__ __forceinline__ uint32_t movm_trans_b16(uint32_t v) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(v));
  return d;
}

// Orientation: tokens are the MMA rows.  Per page (16 tokens):
//   S^T[16 tokens x 8 heads]  = K[16 x 128] . q^T[128 x 8]          (8 k-steps, A = K via ldmatrix)
//   O^T[128 dims x 8 heads]  += V^T[128 x 16] . P^T[16 x 8]          (8 row tiles, A = V via ldmatrix.trans,
//                                                                   B = P^T after an 8x8 movmatrix transpose)
// so both products use all 16 rows of the tile and the accumulator is 32 registers per 8 heads.
template <int NH, bool CONTIG>
__global__ void __launch_bounds__(LOCKS_ATT_WARPS * 32) attend_bf16_kernel(AttParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int x = lane >> 2, t = lane & 3;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int64_t prob = (int64_t)b * p.Hkv + h;
  const int hkv = h / p.kvdiv;   // head of the cache this problem reads
  uint8_t *ring = smem + warp * kAttStages * kAttStage;
  const uint8_t *Kb = reinterpret_cast<const uint8_t *>(p.k);
  const uint8_t *Vb = reinterpret_cast<const uint8_t *>(p.v);
  pdl_trigger();

  // query as the B operand: lane (x, t) holds head x (+8), dims 16 s + 2t.. and 16 s + 8 + 2t..
  uint32_t qb[NH][8][2];
  {
    const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(p.q);
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      const int g = x + 8 * hh;
      const uint32_t *qr = reinterpret_cast<const uint32_t *>(q + ((int64_t)b * p.Hq + h * p.G + g) * LOCKS_D);
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        qb[hh][s][0] = (g < p.G) ? __ldg(qr + 8 * s + t) : 0u;
        qb[hh][s][1] = (g < p.G) ? __ldg(qr + 8 * s + 4 + t) : 0u;
      }
    }
  }
  const float c2 = p.sm_scale * kLog2e;
  pdl_wait();   // page table from the selector, appended K/V rows, sequence lengths
  const int T = p.seq_lens[b];
  const int P = (T + LOCKS_B - 1) / LOCKS_B;
  int npages = p.ids ? p.cnt[prob] : P;
  if (p.ids && (npages < 0 || npages > p.kbud)) {   // a count beyond the table's row: use the row, report it
    if (threadIdx.x == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
    npages = npages < 0 ? 0 : p.kbud;
  }
  const int lo = split * p.pages_per_cta;
  const int hi = min(lo + p.pages_per_cta, npages);

  float oacc[8][NH][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) oacc[i][hh][0] = oacc[i][hh][1] = oacc[i][hh][2] = oacc[i][hh][3] = 0.f;
  float mrun[NH][2], lrun[NH][2];   // per head column 2t, 2t+1 (+8): running max, this lane's partial sum
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) { mrun[hh][0] = mrun[hh][1] = -INFINITY; lrun[hh][0] = lrun[hh][1] = 0.f; }

  // per-lane constants of the 16-byte copies: copy i moves chunk (lane & 15) of token (lane >> 4) + 2 i
  const int tok0 = lane >> 4, ch0 = lane & 15;
  const int64_t goff0 = ((int64_t)tok0 * p.st + ch0 * 8) * 2;       // bytes
  const int64_t gstep = p.st * 4;                                    // two token rows, bytes
  uint32_t sw[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) sw[i] = (uint32_t)(tok0 * 256 + (((ch0 ^ tok0) ^ ((2 * i) & 7)) << 4));

  // page ids and physical blocks of this warp's pages are resolved 32 at a time, one lane each, so the
  // two dependent global loads are paid once per batch instead of once per page
  const int first = lo + warp;
  auto resolve_batch = [&](int jb, int &blk, int &nt) {
    const int idx = first + (jb + lane) * LOCKS_ATT_WARPS;
    blk = 0;
    nt = 0;
    if (idx < hi && !resolve_page(p, b, prob, idx, T, blk, nt)) nt = 0;
  };
  int blk_cur, nt_cur, blk_nxt = 0, nt_nxt = 0;
  resolve_batch(0, blk_cur, nt_cur);

  const uint64_t pol_stream = l2_policy_evict_first();
  auto issue = [&](int j, int stage) -> int {  // j-th page of this warp; returns its valid tokens
    const int block = __shfl_sync(0xffffffffu, blk_cur, j & 31);
    const int ntok = __shfl_sync(0xffffffffu, nt_cur, j & 31);
    uint8_t *kt = ring + stage * kAttStage, *vt = kt + kTile;
    const int64_t base = ((int64_t)block * p.sb + (int64_t)hkv * p.sh) * 2 + goff0;
    const uint8_t *kp = Kb + base, *vp = Vb + base;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t so = sw[i & 3] + 512 * i;
      const bool valid = tok0 + 2 * i < ntok;   // rows past the sequence end are zero-filled
      if (LOCKS_ATT_HINT_LOAD) {   // K and V stream through L2 once: they should not push out the small
                                   // tables (lengths, block table, page ids) every kernel of the step re-reads
        if (CONTIG) {   // token rows are 256 bytes apart: immediate offsets
          cp_async16_hint(kt + so, kp + i * 512, valid, pol_stream);
          cp_async16_hint(vt + so, vp + i * 512, valid, pol_stream);
        } else {
          cp_async16_hint(kt + so, kp + i * gstep, valid, pol_stream);
          cp_async16_hint(vt + so, vp + i * gstep, valid, pol_stream);
        }
      } else if (CONTIG) {
        cp_async16(kt + so, kp + i * 512, valid);
        cp_async16(vt + so, vp + i * 512, valid);
      } else {
        cp_async16(kt + so, kp + i * gstep, valid);
        cp_async16(vt + so, vp + i * gstep, valid);
      }
    }
    cp_async_commit();
    return ntok;
  };

  // ring of kAttStages pages per warp: pages j+1 .. j+kAttStages-1 are in flight while page j is used
  const int npg = (hi > first) ? (hi - first + LOCKS_ATT_WARPS - 1) / LOCKS_ATT_WARPS : 0;   // this warp's pages
  int ntok_ring[kAttStages];
#pragma unroll
  for (int s2 = 0; s2 < kAttStages - 1; ++s2) {
    ntok_ring[s2] = 0;
    if (s2 < npg) ntok_ring[s2] = issue(s2, s2); else cp_async_commit();
  }
  ntok_ring[kAttStages - 1] = 0;
  for (int j = 0; j < npg; ++j) {
    const int stage = j % kAttStages;
    if ((j & 31) == 15) resolve_batch((j & ~31) + 32, blk_nxt, nt_nxt);   // next batch, half a batch early
    {
      const int jn = j + kAttStages - 1;   // refill the slot freed by page j-1
      if (((jn) & 31) == 0 && jn > 0) { blk_cur = blk_nxt; nt_cur = nt_nxt; }
      int nt_new = 0;
      if (jn < npg) nt_new = issue(jn, jn % kAttStages); else cp_async_commit();
#pragma unroll
      for (int s2 = 0; s2 < kAttStages; ++s2) if (s2 == jn % kAttStages) ntok_ring[s2] = nt_new;
    }
    cp_async_wait<kAttStages - 1>();
    int ntok_cur = 0;
#pragma unroll
    for (int s2 = 0; s2 < kAttStages; ++s2) if (s2 == stage) ntok_cur = ntok_ring[s2];
    __syncwarp();
    const uint8_t *kt = ring + stage * kAttStage, *vt = kt + kTile;
    const int ntok = ntok_cur;
    const int m = lane >> 3, rr = lane & 7;
    // ---- S^T = K q^T
    float sacc[NH][4];
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) sacc[hh][0] = sacc[hh][1] = sacc[hh][2] = sacc[hh][3] = 0.f;
    {
      const int tok = (m & 1) * 8 + rr;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const int ch = 2 * s + (m >> 1);
        uint32_t r[4];
        ldsm_x4(r, kt + tok * 256 + ((ch ^ (tok & 7)) << 4));
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) mma_bf16(sacc[hh], r[0], r[1], r[2], r[3], qb[hh][s][0], qb[hh][s][1]);
      }
    }
    // ---- online softmax down the token rows; this lane: tokens x, x + 8, heads 2t, 2t+1 (+8)
    uint32_t pb0[NH], pb1[NH];
    const bool v0ok = x < ntok, v1ok = x + 8 < ntok;
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      float sv[4];
      sv[0] = v0ok ? sacc[hh][0] * c2 : -INFINITY;
      sv[1] = v0ok ? sacc[hh][1] * c2 : -INFINITY;
      sv[2] = v1ok ? sacc[hh][2] * c2 : -INFINITY;
      sv[3] = v1ok ? sacc[hh][3] * c2 : -INFINITY;
      float cm0 = fmaxf(sv[0], sv[2]), cm1 = fmaxf(sv[1], sv[3]);
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        cm0 = fmaxf(cm0, __shfl_xor_sync(0xffffffffu, cm0, o));
        cm1 = fmaxf(cm1, __shfl_xor_sync(0xffffffffu, cm1, o));
      }
      const float mn0 = fmaxf(mrun[hh][0], cm0), mn1 = fmaxf(mrun[hh][1], cm1);
      const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
      const bool moved = (mn0 != mrun[hh][0]) || (mn1 != mrun[hh][1]);
      if (__any_sync(0xffffffffu, moved)) {   // rescale only when some running max rose
        const float a0 = ex2f(mrun[hh][0] - ms0), a1 = ex2f(mrun[hh][1] - ms1);
        lrun[hh][0] *= a0;
        lrun[hh][1] *= a1;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          oacc[i][hh][0] *= a0; oacc[i][hh][2] *= a0;
          oacc[i][hh][1] *= a1; oacc[i][hh][3] *= a1;
        }
      }
      mrun[hh][0] = mn0;
      mrun[hh][1] = mn1;
      const float p00 = ex2f(sv[0] - ms0), p01 = ex2f(sv[1] - ms1), p10 = ex2f(sv[2] - ms0), p11 = ex2f(sv[3] - ms1);
      lrun[hh][0] += p00 + p10;
      lrun[hh][1] += p01 + p11;
      // P^T rows (tokens) -> B fragment (k = tokens 2t, 2t+1 | 8 + 2t.., n = head x)
      pb0[hh] = movm_trans_b16(pack_bf16(p00, p01));
      pb1[hh] = movm_trans_b16(pack_bf16(p10, p11));
    }
    // ---- O^T += V^T P^T
    {
      const int tok = (m >> 1) * 8 + rr;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        const int ch = 2 * mt + (m & 1);
        uint32_t r[4];
        ldsm_x4_trans(r, vt + tok * 256 + ((ch ^ (tok & 7)) << 4));
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) mma_bf16(oacc[mt][hh], r[0], r[1], r[2], r[3], pb0[hh], pb1[hh]);
      }
    }
    __syncwarp();
  }
  cp_async_wait<0>();
#pragma unroll
  for (int hh = 0; hh < NH; ++hh)
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) lrun[hh][c] += __shfl_xor_sync(0xffffffffu, lrun[hh][c], o);
  __syncthreads();  // every warp is done with its ring: reuse it for the merge
  float *wo = reinterpret_cast<float *>(ring);          // [16 heads][128] fp32
  float *wm = wo + 16 * LOCKS_D, *wl = wm + 16;          // [16], [16]
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int row = 8 * hh + 2 * t + c;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        wo[row * LOCKS_D + 16 * mt + x] = oacc[mt][hh][c];
        wo[row * LOCKS_D + 16 * mt + 8 + x] = oacc[mt][hh][2 + c];
      }
      if (x == 0) { wm[row] = mrun[hh][c]; wl[row] = lrun[hh][c]; }
    }
  }
  __syncthreads();
  if (p.cluster) {
    // The splits of this (request, KV head) are the CTAs of one cluster.  Each CTA first folds its warps into
    // one unnormalised partial in its own shared memory; after a cluster barrier CTA r produces a slice of the
    // problem's G x 128 outputs by reading every CTA's partial through distributed shared memory; a second
    // barrier keeps every CTA's memory alive until its peers are done.  No partial leaves the SMs.
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    constexpr int NT = LOCKS_ATT_WARPS * 32;
    // the CTA's partial replaces warp 0's in place (element e is read and written by one thread only); its
    // (max, sum) go to the idle tail of warp 1's ring, because other threads still read warp 0's
    float *co = reinterpret_cast<float *>(smem);
    float *cm = reinterpret_cast<float *>(smem + kAttStages * kAttStage) + 16 * LOCKS_D + 32, *cl = cm + 16;
    for (int e = threadIdx.x; e < p.G * LOCKS_D; e += NT) {
      const int g = e / LOCKS_D, dim = e - g * LOCKS_D;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < LOCKS_ATT_WARPS; ++w)
        M = fmaxf(M, reinterpret_cast<const float *>(smem + w * kAttStages * kAttStage)[16 * LOCKS_D + g]);
      float L = 0.f, o = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int w = 0; w < LOCKS_ATT_WARPS; ++w) {
          const float *ww = reinterpret_cast<const float *>(smem + w * kAttStages * kAttStage);
          const float sc = ex2f(ww[16 * LOCKS_D + g] - M);
          L += ww[16 * LOCKS_D + 16 + g] * sc;
          o += ww[g * LOCKS_D + dim] * sc;
        }
      }
      co[e] = o;
      if (dim == 0) { cm[g] = M; cl[g] = L; }
    }
    cluster.sync();
    const int nout = p.G * LOCKS_D, per = (nout + p.splits - 1) / p.splits;
    const int e1 = min(nout, (split + 1) * per);
    for (int e = split * per + threadIdx.x; e < e1; e += NT) {
      const int g = e / LOCKS_D;
      float mv[16], lv[16], ov[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        mv[c] = -INFINITY; lv[c] = 0.f; ov[c] = 0.f;
        if (c < p.splits) {
          mv[c] = cluster.map_shared_rank(cm, c)[g];
          lv[c] = cluster.map_shared_rank(cl, c)[g];
          ov[c] = cluster.map_shared_rank(co, c)[e];
        }
      }
      float M = -INFINITY;
#pragma unroll
      for (int c = 0; c < 16; ++c) M = fmaxf(M, mv[c]);
      float L = 0.f, o = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const float sc = ex2f(mv[c] - M);
          L = fmaf(lv[c], sc, L);
          o = fmaf(ov[c], sc, o);
        }
        o /= L;
      }
      const int64_t row = (int64_t)b * p.Hq + h * p.G + g;
      reinterpret_cast<__nv_bfloat16 *>(p.out)[row * LOCKS_D + (e - g * LOCKS_D)] = __float2bfloat16_rn(o);
      if (p.lse && e == g * LOCKS_D) p.lse[row] = (M > -INFINITY) ? (M + log2f(L)) * kLn2 : -INFINITY;
    }
    cluster.sync();
    return;
  }
  for (int e = threadIdx.x; e < p.G * LOCKS_D; e += LOCKS_ATT_WARPS * 32) {
    const int g = e / LOCKS_D, dim = e - g * LOCKS_D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < LOCKS_ATT_WARPS; ++w)
      M = fmaxf(M, reinterpret_cast<const float *>(smem + w * kAttStages * kAttStage)[16 * LOCKS_D + g]);
    float L = 0.f, o = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < LOCKS_ATT_WARPS; ++w) {
        const float *ww = reinterpret_cast<const float *>(smem + w * kAttStages * kAttStage);
        const float sc = ex2f(ww[16 * LOCKS_D + g] - M);
        L += ww[16 * LOCKS_D + 16 + g] * sc;
        o += ww[g * LOCKS_D + dim] * sc;
      }
      o /= L;
    }
    const int hq = h * p.G + g;
    const float lse2 = (M > -INFINITY) ? M + log2f(L) : -INFINITY;
    if (p.splits == 1) {
      reinterpret_cast<__nv_bfloat16 *>(p.out)[((int64_t)b * p.Hq + hq) * LOCKS_D + dim] = __float2bfloat16_rn(o);
      if (p.lse && dim == 0) p.lse[(int64_t)b * p.Hq + hq] = lse2 * kLn2;
    } else {
      const int64_t slot = ((int64_t)b * p.Hq + hq) * p.splits + split;
      p.part_o[slot * LOCKS_D + dim] = o;
      if (dim == 0) p.part_lse[slot] = lse2;
    }
  }
  if (p.splits == 1 || !p.fused_merge) return;
  // the last CTA of this (request, KV head) to arrive merges the splits' partials by log-sum-exp
  __shared__ int sh_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) sh_last = (atomicAdd(&p.done[prob], 1) == p.splits - 1);
  __syncthreads();
  if (!sh_last) return;
  __threadfence();
  // weights of the splits: sh_w[g][s] = 2^(lse_s - max), then normalised by their sum
  float *sh_w = reinterpret_cast<float *>(smem);   // [G][splits] <= 16 x 64 floats, the rings are idle now
  constexpr int NT = LOCKS_ATT_WARPS * 32;
  for (int e = threadIdx.x; e < p.G * p.splits; e += NT) {
    const int g = e / p.splits, s2 = e - g * p.splits;
    sh_w[e] = __ldcg(p.part_lse + ((int64_t)b * p.Hq + h * p.G + g) * p.splits + s2);
  }
  __syncthreads();
  if (threadIdx.x < p.G) {
    float *w = sh_w + threadIdx.x * p.splits;
    float M = -INFINITY;
    for (int s2 = 0; s2 < p.splits; ++s2) M = fmaxf(M, w[s2]);
    float L = 0.f;
    for (int s2 = 0; s2 < p.splits; ++s2) { const float v = (M > -INFINITY) ? ex2f(w[s2] - M) : 0.f; w[s2] = v; L += v; }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int s2 = 0; s2 < p.splits; ++s2) w[s2] *= inv;
    if (p.lse) p.lse[(int64_t)b * p.Hq + h * p.G + threadIdx.x] = (M > -INFINITY) ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < p.G * (LOCKS_D / 4); e += NT) {   // four dims per thread, loads batched by 4 splits
    const int g = e / (LOCKS_D / 4), d4 = e - g * (LOCKS_D / 4);
    const int64_t row = (int64_t)b * p.Hq + h * p.G + g;
    const float4 *po = reinterpret_cast<const float4 *>(p.part_o + row * p.splits * LOCKS_D) + d4;
    const float *w = sh_w + g * p.splits;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < p.splits; s0 += 4) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        v[u] = (s0 + u < p.splits) ? __ldcg(po + (int64_t)(s0 + u) * (LOCKS_D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float ww = (s0 + u < p.splits) ? w[s0 + u] : 0.f;
        acc.x += ww * v[u].x; acc.y += ww * v[u].y; acc.z += ww * v[u].z; acc.w += ww * v[u].w;
      }
    }
    __nv_bfloat162 *dst = reinterpret_cast<__nv_bfloat162 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + row * LOCKS_D + 4 * d4);
    dst[0] = __floats2bfloat162_rn(acc.x, acc.y);
    dst[1] = __floats2bfloat162_rn(acc.z, acc.w);
  }
  if (threadIdx.x == 0) p.done[prob] = 0;   // ready for the next launch
}

// Plain fp32-arithmetic path for any element type (the fp32 parity configuration).
template <typename T>
__global__ void __launch_bounds__(128) attend_generic_kernel(AttParams p) {
  __shared__ float so[4][LOCKS_D];
  __shared__ float sm[4], sl[4];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int split = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const int h = hq / p.G;
  pdl_wait();
  const int64_t prob = (int64_t)b * p.Hkv + h;
  const int Tn = p.seq_lens[b];
  const int P = (Tn + p.B - 1) / p.B;
  int npages = p.ids ? p.cnt[prob] : P;
  if (p.ids && (npages < 0 || npages > p.kbud)) {
    if (threadIdx.x == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
    npages = npages < 0 ? 0 : p.kbud;
  }
  const int lo = split * p.pages_per_cta, hi = min(lo + p.pages_per_cta, npages);
  const T *K = reinterpret_cast<const T *>(p.k), *V = reinterpret_cast<const T *>(p.v), *Q = reinterpret_cast<const T *>(p.q);
  float qv[4], o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int u = 0; u < 4; ++u) qv[u] = ldf<T>(Q, ((int64_t)b * p.Hq + hq) * LOCKS_D + lane * 4 + u);
  float m = -INFINITY, l = 0.f;
  const float c2 = p.sm_scale * kLog2e;
  for (int idx = lo + warp; idx < hi; idx += 4) {
    int block, ntok;
    if (!resolve_page(p, b, prob, idx, Tn, block, ntok)) continue;
    const int64_t base = (int64_t)block * p.sb + (int64_t)(h / p.kvdiv) * p.sh;
    for (int i = 0; i < ntok; ++i) {
      float s = 0.f;
#pragma unroll
      for (int u = 0; u < 4; ++u) s += qv[u] * ldf<T>(K, base + (int64_t)i * p.st + lane * 4 + u);
      s = warp_sum(s) * c2;
      const float mn = fmaxf(m, s);
      const float alpha = exp2f(m - mn), pw = exp2f(s - mn);
      l = l * alpha + pw;
#pragma unroll
      for (int u = 0; u < 4; ++u) o[u] = o[u] * alpha + pw * ldf<T>(V, base + (int64_t)i * p.st + lane * 4 + u);
      m = mn;
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) so[warp][lane * 4 + u] = o[u];
  if (lane == 0) { sm[warp] = m; sl[warp] = l; }
  __syncthreads();
  const int dim = threadIdx.x;
  float M = fmaxf(fmaxf(sm[0], sm[1]), fmaxf(sm[2], sm[3]));
  float L = 0.f, acc = 0.f;
  if (M > -INFINITY) {
    for (int w = 0; w < 4; ++w) {
      const float sc = exp2f(sm[w] - M);
      L += sl[w] * sc;
      acc += so[w][dim] * sc;
    }
    acc /= L;
  }
  const float lse2 = (M > -INFINITY) ? M + log2f(L) : -INFINITY;
  if (p.splits == 1) {
    stf<T>(reinterpret_cast<T *>(p.out), ((int64_t)b * p.Hq + hq) * LOCKS_D + dim, acc);
    if (p.lse && dim == 0) p.lse[(int64_t)b * p.Hq + hq] = lse2 * kLn2;
  } else {
    const int64_t slot = ((int64_t)b * p.Hq + hq) * p.splits + split;
    p.part_o[slot * LOCKS_D + dim] = acc;
    if (dim == 0) p.part_lse[slot] = lse2;
  }
}

// Merge of the split-K partials of one query head: 128 threads = 4 split slices x 32 four-dim columns.
template <typename T>
__global__ void __launch_bounds__(128) attend_merge_kernel(const float *part_o, const float *part_lse, int splits,
                                                           T *out, float *lse, int Hq) {
  __shared__ float sw[LOCKS_ATT_MAX_SPLITS];
  __shared__ float4 sacc[4][32];
  const int hq = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
  pdl_wait();
  const int64_t row = (int64_t)b * Hq + hq;
  for (int s = tid; s < splits; s += 128) sw[s] = part_lse[row * splits + s];
  __syncthreads();
  if (tid < 32) {
    float M = -INFINITY;
    for (int s = lane; s < splits; s += 32) M = fmaxf(M, sw[s]);
    M = warp_max(M);
    float L = 0.f;
    for (int s = lane; s < splits; s += 32) { const float w = (M > -INFINITY) ? exp2f(sw[s] - M) : 0.f; sw[s] = w; L += w; }
    L = warp_sum(L);
    const float inv = L > 0.f ? 1.f / L : 0.f;
    __syncwarp();
    for (int s = lane; s < splits; s += 32) sw[s] *= inv;
    if (lse && lane == 0) lse[row] = (M > -INFINITY) ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
  __syncthreads();
  const int sl = tid >> 5;
  const float4 *po = reinterpret_cast<const float4 *>(part_o + row * splits * LOCKS_D) + lane;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = sl; s0 < splits; s0 += 16) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      v[u] = (s0 + 4 * u < splits) ? __ldcg(po + (int64_t)(s0 + 4 * u) * (LOCKS_D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float w = (s0 + 4 * u < splits) ? sw[s0 + 4 * u] : 0.f;
      acc.x += w * v[u].x; acc.y += w * v[u].y; acc.z += w * v[u].z; acc.w += w * v[u].w;
    }
  }
  sacc[sl][lane] = acc;
  __syncthreads();
  if (sl == 0) {
    const float4 a1 = sacc[1][lane], a2 = sacc[2][lane], a3 = sacc[3][lane];
    acc.x += a1.x + a2.x + a3.x; acc.y += a1.y + a2.y + a3.y; acc.z += a1.z + a2.z + a3.z; acc.w += a1.w + a2.w + a3.w;
    stf<T>(out, row * LOCKS_D + 4 * lane + 0, acc.x);
    stf<T>(out, row * LOCKS_D + 4 * lane + 1, acc.y);
    stf<T>(out, row * LOCKS_D + 4 * lane + 2, acc.z);
    stf<T>(out, row * LOCKS_D + 4 * lane + 3, acc.w);
  }
}

// Merge of the attention partials of several shards of one sequence (each normalised over its own pages, with
// its natural-log lse): out = sum_r w_r o_r, w_r = exp(lse_r - LSE), LSE = log sum_r exp(lse_r).
template <typename T>
__global__ void __launch_bounds__(LOCKS_D) merge_shards_kernel(const T *part_out, const float *part_lse, int nparts, int rows,
                                                              T *out, float *lse) {
  const int row = blockIdx.x, dim = threadIdx.x;
  float M = -INFINITY;
  for (int r = 0; r < nparts; ++r) M = fmaxf(M, part_lse[(int64_t)r * rows + row]);
  float L = 0.f, acc = 0.f;
  if (M > -INFINITY) {
    for (int r = 0; r < nparts; ++r) {
      const float l = part_lse[(int64_t)r * rows + row];
      if (l == -INFINITY) continue;
      const float w = __expf(l - M);
      L += w;
      acc += w * ldf<T>(part_out, ((int64_t)r * rows + row) * LOCKS_D + dim);
    }
    acc /= L;
  }
  stf<T>(out, (int64_t)row * LOCKS_D + dim, acc);
  if (lse && dim == 0) lse[row] = M > -INFINITY ? M + __logf(L) : -INFINITY;
}

}  // namespace

int locks_launch_merge_shards(locks_ctx *c, const void *part_out, const float *part_lse, int nparts, int batch, void *out,
                              float *lse, cudaStream_t st) {
  const int rows = batch * c->cfg.num_q_heads;
  if (c->cfg.q_dtype == LOCKS_BF16)
    merge_shards_kernel<__nv_bfloat16><<<rows, LOCKS_D, 0, st>>>(reinterpret_cast<const __nv_bfloat16 *>(part_out), part_lse, nparts,
                                                                rows, reinterpret_cast<__nv_bfloat16 *>(out), lse);
  else
    merge_shards_kernel<float><<<rows, LOCKS_D, 0, st>>>(reinterpret_cast<const float *>(part_out), part_lse, nparts, rows,
                                                        reinterpret_cast<float *>(out), lse);
  return locks_check_launch(c);
}

int locks_launch_attend(locks_ctx *c, const void *q, const locks_kv *kv, int batch, const int32_t *ids,
                        const int32_t *cnt, void *out, float *lse, cudaStream_t st) {
  AttParams p;
  p.q = q; p.k = kv->k; p.v = kv->v; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.ids = ids; p.cnt = cnt;
  p.part_o = c->att_o; p.part_lse = c->att_lse; p.out = out; p.lse = lse; p.status = c->status;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G; p.Pmax = c->Pmax;
  p.kbud = c->k; p.num_blocks = kv->num_blocks; p.sm_scale = c->cfg.sm_scale; p.B = c->B; p.kvdiv = 1;
  if (c->cfg.combine == LOCKS_COMBINE_PER_HEAD && ids) {   // one page table per query head: groups of one
    p.kvdiv = p.G; p.Hkv = p.Hq; p.G = 1;
  }
  const bool dense = ids == nullptr;
  // one wave: as many splits per problem as resident CTA slots allow, at least one page per warp
  const int npages = dense ? c->Pmax : c->k;
  int slots = c->num_sms * LOCKS_ATT_CTAS_PER_SM;
  if (slots > LOCKS_ATT_SLOT_BOUND) slots = LOCKS_ATT_SLOT_BOUND;
  int splits = slots / (batch * p.Hkv);
  const int most = (npages + LOCKS_ATT_WARPS - 1) / LOCKS_ATT_WARPS;
  if (splits > most) splits = most;
  if (splits > LOCKS_ATT_MAX_SPLITS) splits = LOCKS_ATT_MAX_SPLITS;
  if (splits < 1) splits = 1;
  // With clearly more problems than SMs every SM streams for several CTAs already: splitting a problem in
  // two only adds the merge (config 2, 256 problems: -1.5 to -2 us per step with one CTA per problem)
  if (!dense && 2 * batch * p.Hkv >= 3 * c->num_sms) splits = 1;
  p.pages_per_cta = (npages + splits - 1) / splits;
  p.splits = (npages + p.pages_per_cta - 1) / p.pages_per_cta;
  p.done = c->att_done;
  // a single CTA merging many splits of many heads is a serial tail: beyond 64 (head, split) pairs use the
  // parallel merge kernel instead
  p.fused_merge = (p.G * p.splits <= 64) ? 1 : 0;
  // Preferred: the splits of a problem as one thread-block cluster (2, 4, 8 or 16 CTAs) that merges through
  // distributed shared memory, as long as a CTA then has at most 8 pages per warp to stream.
  p.cluster = 0;
  if (c->att_cluster_max < 0) {   // largest cluster of this kernel the device can place (probed once)
    c->att_cluster_max = 0;
    cudaFuncSetAttribute(attend_bf16_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
    cudaFuncSetAttribute(attend_bf16_kernel<1, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    for (int cs = 16; cs >= 2 && c->att_cluster_max == 0; cs /= 2) {
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3(cs, 1, 1);
      lc.blockDim = dim3(LOCKS_ATT_WARPS * 32);
      lc.dynamicSmemBytes = kAttSmem;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.attrs = at;
      lc.numAttrs = 1;
      int nclusters = 0;
      if (cudaOccupancyMaxActiveClusters(&nclusters, attend_bf16_kernel<1, true>, &lc) == cudaSuccess && nclusters > 0)
        c->att_cluster_max = cs;
    }
    (void)cudaGetLastError();   // a refused probe is not an error of this call
  }
  if (c->cfg.kv_dtype == LOCKS_BF16 && c->B == LOCKS_B && splits >= 2 && c->att_cluster_max >= 2) {
    int cs = 2;
    while (cs * 2 <= splits && cs * 2 <= c->att_cluster_max) cs *= 2;
    const int ppc = (npages + cs - 1) / cs;
    if (ppc <= 8 * LOCKS_ATT_WARPS && (npages + ppc - 1) / ppc == cs) {
      p.cluster = 1;
      p.pages_per_cta = ppc;
      p.splits = cs;
      p.fused_merge = 1;   // no merge launch follows
    }
  }
  const bool bf = c->cfg.kv_dtype == LOCKS_BF16 && c->B == LOCKS_B;   // tensor-core kernel: bf16 cache, 16-token pages
  if (bf) {
    if (locks_attrs_needed(LOCKS_ATTR_ATTEND)) {
      cudaFuncSetAttribute(attend_bf16_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
      cudaFuncSetAttribute(attend_bf16_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
      cudaFuncSetAttribute(attend_bf16_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
      cudaFuncSetAttribute(attend_bf16_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
      cudaFuncSetAttribute(attend_bf16_kernel<1, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      cudaFuncSetAttribute(attend_bf16_kernel<2, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      cudaFuncSetAttribute(attend_bf16_kernel<1, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      cudaFuncSetAttribute(attend_bf16_kernel<2, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    }
    dim3 grid(p.splits, p.Hkv, batch);
    const bool contig = kv->stride_token == LOCKS_D;
    const dim3 blk(LOCKS_ATT_WARPS * 32);
    if (p.cluster) {
      if (p.G <= 8) {
        if (contig) locks_launch_pdl_cluster(attend_bf16_kernel<1, true>, grid, blk, kAttSmem, p.splits, st, p);
        else locks_launch_pdl_cluster(attend_bf16_kernel<1, false>, grid, blk, kAttSmem, p.splits, st, p);
      } else {
        if (contig) locks_launch_pdl_cluster(attend_bf16_kernel<2, true>, grid, blk, kAttSmem, p.splits, st, p);
        else locks_launch_pdl_cluster(attend_bf16_kernel<2, false>, grid, blk, kAttSmem, p.splits, st, p);
      }
    } else if (p.G <= 8) {
      if (contig) locks_launch_pdl(attend_bf16_kernel<1, true>, grid, blk, kAttSmem, st, p);
      else locks_launch_pdl(attend_bf16_kernel<1, false>, grid, blk, kAttSmem, st, p);
    } else {
      if (contig) locks_launch_pdl(attend_bf16_kernel<2, true>, grid, blk, kAttSmem, st, p);
      else locks_launch_pdl(attend_bf16_kernel<2, false>, grid, blk, kAttSmem, st, p);
    }
  } else {
    dim3 grid(p.splits, p.Hq, batch);
    if (c->cfg.kv_dtype == LOCKS_BF16) locks_launch_pdl(attend_generic_kernel<__nv_bfloat16>, grid, dim3(128), 0, st, p);
    else locks_launch_pdl(attend_generic_kernel<float>, grid, dim3(128), 0, st, p);
  }
  int rc = locks_check_launch(c);
  if (rc != LOCKS_OK || p.splits == 1 || (bf && p.fused_merge)) return rc;
  dim3 mg(p.Hq, batch);
  if (c->cfg.kv_dtype == LOCKS_BF16) locks_launch_pdl(attend_merge_kernel<__nv_bfloat16>, mg, dim3(128), 0, st, (const float *)c->att_o,
                           (const float *)c->att_lse, p.splits, reinterpret_cast<__nv_bfloat16 *>(out), lse, p.Hq);
  else locks_launch_pdl(attend_merge_kernel<float>, mg, dim3(128), 0, st, (const float *)c->att_o,
                        (const float *)c->att_lse, p.splits, reinterpret_cast<float *>(out), lse, p.Hq);
  return locks_check_launch(c);
}

// ------------------------------------------------------------------------------------------------
// Sparse attention for callers that cannot allocate device memory.
//
// The split-K partials and the split-arrival counters of attend_bf16_kernel normally live in the
// workspace the caller allocates for locks_create().  This variant keeps them in a fixed array that is
// part of the library image instead, so nothing has to be allocated at all.
// ------------------------------------------------------------------------------------------------

namespace {

constexpr int kNoAllocMaxRows = LOCKS_NOALLOC_MAX_ROWS;          // batch * Hq
constexpr int kNoAllocMaxSplits = LOCKS_NOALLOC_MAX_SPLITS;
constexpr size_t kNoAllocO = (size_t)kNoAllocMaxRows * kNoAllocMaxSplits * LOCKS_D * sizeof(float);
constexpr size_t kNoAllocLse = (size_t)kNoAllocMaxRows * kNoAllocMaxSplits * sizeof(float);
constexpr size_t kNoAllocDone = (size_t)kNoAllocMaxRows * sizeof(int32_t);   // >= batch * Hkv
constexpr size_t kNoAllocBytes = kNoAllocO + kNoAllocLse + kNoAllocDone + 256;

// About 2.1 MB held by every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

struct NoAllocDevice {
  unsigned char *scratch;   // device address of g_noalloc_scratch on this device (not the host symbol!)
  int num_sms;
  bool ready;
};
NoAllocDevice g_noalloc_dev[64] = {};
std::mutex g_noalloc_mu;   // guards the per-device set-up (two host threads may make a device's first call)

}  // namespace

extern "C" int locks_sparse_attend_noalloc(const locks_config *cfg, const void *q, const locks_kv *kv, int batch,
                                           const int32_t *page_ids, const int32_t *page_count, void *out, float *lse,
                                           locks_stream stream) {
  if (!cfg || !q || !kv || !out || !kv->k || !kv->v || !kv->block_table || !kv->seq_lens) return LOCKS_ERR_INVALID_ARG;
  if ((page_ids == nullptr) != (page_count == nullptr) || batch <= 0 || kv->num_blocks <= 0) return LOCKS_ERR_INVALID_ARG;
  if (cfg->num_q_heads <= 0 || cfg->num_kv_heads <= 0 || cfg->num_q_heads % cfg->num_kv_heads) return LOCKS_ERR_INVALID_ARG;
  if (cfg->max_pages_per_seq <= 0 || cfg->budget_tokens <= 0 || !(cfg->sm_scale > 0.f)) return LOCKS_ERR_INVALID_ARG;
  if (cfg->head_dim != LOCKS_D || cfg->page_size != LOCKS_B || cfg->kv_dtype != LOCKS_BF16 || cfg->q_dtype != LOCKS_BF16)
    return LOCKS_ERR_UNSUPPORTED;
  const int G = cfg->num_q_heads / cfg->num_kv_heads;
  if (G > 16) return LOCKS_ERR_UNSUPPORTED;
  if ((kv->stride_block | kv->stride_head | kv->stride_token) % 8 || kv->stride_token < LOCKS_D) return LOCKS_ERR_INVALID_ARG;
  if (((uintptr_t)kv->k | (uintptr_t)kv->v | (uintptr_t)q) % 16) return LOCKS_ERR_INVALID_ARG;
  // the built-in scratch bounds the problem: reject anything that would not fit
  if ((int64_t)batch * cfg->num_q_heads > kNoAllocMaxRows) return LOCKS_ERR_TOO_LARGE;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LOCKS_ERR_CUDA;
  NoAllocDevice &nd = g_noalloc_dev[dev];
  std::unique_lock<std::mutex> setup_lock(g_noalloc_mu);
  if (!nd.ready) {
    // first call on this device: ask the runtime where the array lives on the CURRENT device
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return LOCKS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&nd.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LOCKS_ERR_CUDA;
    cudaFuncSetAttribute(attend_bf16_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
    cudaFuncSetAttribute(attend_bf16_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
    cudaFuncSetAttribute(attend_bf16_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
    cudaFuncSetAttribute(attend_bf16_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
    nd.scratch = reinterpret_cast<unsigned char *>(ptr);
    nd.ready = true;
  }
  setup_lock.unlock();
  cudaStream_t st = (cudaStream_t)stream;
  AttParams p;
  p.q = q; p.k = kv->k; p.v = kv->v; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.ids = page_ids; p.cnt = page_count;
  p.part_o = reinterpret_cast<float *>(nd.scratch);
  p.part_lse = reinterpret_cast<float *>(nd.scratch + kNoAllocO);
  p.done = reinterpret_cast<int32_t *>(nd.scratch + kNoAllocO + kNoAllocLse);
  p.status = reinterpret_cast<int32_t *>(nd.scratch + kNoAllocO + kNoAllocLse + kNoAllocDone);
  p.out = out; p.lse = lse;
  p.batch = batch; p.Hq = cfg->num_q_heads; p.Hkv = cfg->num_kv_heads; p.G = G; p.Pmax = cfg->max_pages_per_seq;
  p.kbud = (cfg->budget_tokens + LOCKS_B - 1) / LOCKS_B; p.num_blocks = kv->num_blocks; p.sm_scale = cfg->sm_scale; p.B = LOCKS_B; p.kvdiv = 1;
  const int npages = page_ids ? p.kbud : p.Pmax;
  int splits = nd.num_sms * LOCKS_ATT_CTAS_PER_SM / (batch * p.Hkv);
  const int most = (npages + LOCKS_ATT_WARPS - 1) / LOCKS_ATT_WARPS;
  if (splits > most) splits = most;
  if (splits > kNoAllocMaxSplits) splits = kNoAllocMaxSplits;
  if (splits < 1) splits = 1;
  p.pages_per_cta = (npages + splits - 1) / splits;
  p.splits = (npages + p.pages_per_cta - 1) / p.pages_per_cta;
  p.fused_merge = 1;
  p.cluster = 0;
  // the array keeps whatever the last call left: the arrival counters and the status word must start at zero
  if (cudaMemsetAsync(p.done, 0, kNoAllocDone + 256, st) != cudaSuccess) return LOCKS_ERR_CUDA;
  dim3 grid(p.splits, p.Hkv, batch);
  const bool contig = kv->stride_token == LOCKS_D;
  if (G <= 8) {
    if (contig) attend_bf16_kernel<1, true><<<grid, LOCKS_ATT_WARPS * 32, kAttSmem, st>>>(p);
    else attend_bf16_kernel<1, false><<<grid, LOCKS_ATT_WARPS * 32, kAttSmem, st>>>(p);
  } else {
    if (contig) attend_bf16_kernel<2, true><<<grid, LOCKS_ATT_WARPS * 32, kAttSmem, st>>>(p);
    else attend_bf16_kernel<2, false><<<grid, LOCKS_ATT_WARPS * 32, kAttSmem, st>>>(p);
  }
  return cudaPeekAtLastError() == cudaSuccess ? LOCKS_OK : LOCKS_ERR_CUDA;
}
