// Diagnostics of the selector (App. B of the paper, "microscope"): the exact-LSE arm and the selection
// fidelity metrics measured against it.
//
//   exact page log-mass (Lemma 1(ii)):  s_j(q_g) = log sum_{i in P_j, i < T} exp(q_g . k_i / sqrt(d))
//
// exact_bf16_kernel reads every K page of the cache (4 KB per (page, KV head): half of what dense attention
// reads) and writes s_j for ALL pages 0..P-1 (the last page over its valid tokens) in the layout of the
// estimated scores, plus one partial (max, sum exp) over the candidate pages 1..P-2 per (head, CTA), so that
// the regular selector kernel ranks them: exact-LSE selection under the same share-average combine, the
// ceiling the paper calls "Oracle".  exact_generic_kernel is the plain fp32 path for fp32 caches.
//
//   quality_kernel: per (request, KV head), mean over the group's heads, all from the exact masses:
//     gamma    total attention mass captured by a page set A:  sum_{j in A} e^{s_j} / sum_{j < P} e^{s_j}
//     gamma_c  contested mass captured: the always-kept pages (0 and P-1) removed from numerator and denominator
//     recall   |A n R| / |R| over the candidate pages of A and of a reference set R (the exact ranking's)
//     needle   of the marked (carrier) pages that R keeps, the fraction A keeps too
#include "locks_internal.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kExWarps = 4;
constexpr int kExPagesPerCta = 64;                      // 16 pages per warp
constexpr int kExStages = 2;
constexpr int kExTile = LOCKS_B * LOCKS_D * 2;          // one K tile, bf16
constexpr int kExSmem = kExWarps * kExStages * kExTile; // 32 KB

struct ExactParams {
  const void *q, *k;
  int64_t sb, sh, st;
  const int32_t *block_table, *seq_lens;
  float *shat;
  float2 *part;
  int32_t *status;
  int batch, Hq, Hkv, G, Pmax, max_groups, num_blocks, kbud;
  float sm_scale;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// online (max, sum) update in the natural-log domain
__device__ __forceinline__ void lse_push(float &m, float &s, float v) {
  if (v == -INFINITY) return;
  const float nm = fmaxf(m, v);
  s = s * __expf(m - nm) + __expf(v - nm);
  m = nm;
}

template <int NH>
__global__ void __launch_bounds__(kExWarps * 32) exact_bf16_kernel(ExactParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ float2 red[kExWarps][16];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int x = lane >> 2, t = lane & 3;
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  uint8_t *ring = smem + warp * kExStages * kExTile;
  const uint8_t *Kb = reinterpret_cast<const uint8_t *>(p.k);
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
  pdl_wait();
  const int T = p.seq_lens[b];
  const int P = (T + LOCKS_B - 1) / LOCKS_B;
  const int lo = chunk * kExPagesPerCta, hi = min(lo + kExPagesPerCta, P);
  // this warp's pages: lo + warp + 4 j, j < 16; lane j resolves page j's block
  const int mypage = lo + warp + kExWarps * lane;
  int blk = 0;
  if (lane < kExPagesPerCta / kExWarps && mypage < hi) {
    blk = p.block_table[(int64_t)b * p.Pmax + mypage];
    if (blk < 0 || blk >= p.num_blocks) { set_status(p.status, LOCKS_ERR_BAD_BLOCK); blk = -1; }
  }
  const int npg = hi > lo + warp ? (hi - lo - warp + kExWarps - 1) / kExWarps : 0;
  const int tok0 = lane >> 4, ch0 = lane & 15;
  const int64_t goff0 = ((int64_t)tok0 * p.st + ch0 * 8) * 2;
  const int64_t gstep = p.st * 4;
  uint32_t sw[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) sw[i] = (uint32_t)(tok0 * 256 + (((ch0 ^ tok0) ^ ((2 * i) & 7)) << 4));
  auto issue = [&](int j, int stage) {
    const int block = __shfl_sync(0xffffffffu, blk, j);
    const int page = lo + warp + kExWarps * j;
    const int ntok = block < 0 ? 0 : min(LOCKS_B, T - page * LOCKS_B);
    uint8_t *kt = ring + stage * kExTile;
    const uint8_t *kp = Kb + ((int64_t)max(block, 0) * p.sb + (int64_t)h * p.sh) * 2 + goff0;
#pragma unroll
    for (int i = 0; i < 8; ++i) cp_async16(kt + sw[i & 3] + 512 * i, kp + i * gstep, tok0 + 2 * i < ntok);
    cp_async_commit();
  };
  float pm[NH][2], ps[NH][2];   // candidate partial of heads 2t, 2t+1 (+8), kept by the lanes x == 0
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) { pm[hh][0] = pm[hh][1] = -INFINITY; ps[hh][0] = ps[hh][1] = 0.f; }
  if (npg > 0) issue(0, 0); else cp_async_commit();
  for (int j = 0; j < npg; ++j) {
    const int stage = j % kExStages;
    if (j + 1 < npg) issue(j + 1, (j + 1) % kExStages); else cp_async_commit();
    cp_async_wait<kExStages - 1>();
    __syncwarp();
    const int page = lo + warp + kExWarps * j;
    const int block = __shfl_sync(0xffffffffu, blk, j);
    const int ntok = block < 0 ? 0 : min(LOCKS_B, T - page * LOCKS_B);
    const uint8_t *kt = ring + stage * kExTile;
    const int m = lane >> 3, rr = lane & 7;
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
    const bool v0ok = x < ntok, v1ok = x + 8 < ntok;
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      const float s0 = v0ok ? sacc[hh][0] * c2 : -INFINITY, s1 = v0ok ? sacc[hh][1] * c2 : -INFINITY;
      const float s2 = v1ok ? sacc[hh][2] * c2 : -INFINITY, s3 = v1ok ? sacc[hh][3] * c2 : -INFINITY;
      float cm0 = fmaxf(s0, s2), cm1 = fmaxf(s1, s3);
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        cm0 = fmaxf(cm0, __shfl_xor_sync(0xffffffffu, cm0, o));
        cm1 = fmaxf(cm1, __shfl_xor_sync(0xffffffffu, cm1, o));
      }
      const float ms0 = cm0 == -INFINITY ? 0.f : cm0, ms1 = cm1 == -INFINITY ? 0.f : cm1;
      float e0 = ex2f(s0 - ms0) + ex2f(s2 - ms0), e1 = ex2f(s1 - ms1) + ex2f(s3 - ms1);
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        e0 += __shfl_xor_sync(0xffffffffu, e0, o);
        e1 += __shfl_xor_sync(0xffffffffu, e1, o);
      }
      if (x == 0 && ntok > 0) {
        const float v0 = (cm0 + log2f(e0)) * kLn2, v1 = (cm1 + log2f(e1)) * kLn2;
        const int g0 = 8 * hh + 2 * t;
        float *dst = p.shat + ((int64_t)b * p.Hq + h * p.G + g0) * p.Pmax + page;
        if (g0 < p.G) dst[0] = v0;
        if (g0 + 1 < p.G) dst[p.Pmax] = v1;
        if (page >= 1 && page <= P - 2) { lse_push(pm[hh][0], ps[hh][0], v0); lse_push(pm[hh][1], ps[hh][1], v1); }
      }
    }
    __syncwarp();
  }
  cp_async_wait<0>();
  // one partial per (head, CTA): merge the four warps
  if (x == 0) {
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      red[warp][8 * hh + 2 * t] = make_float2(pm[hh][0], ps[hh][0]);
      red[warp][8 * hh + 2 * t + 1] = make_float2(pm[hh][1], ps[hh][1]);
    }
  }
  __syncthreads();
  if (threadIdx.x < p.G && threadIdx.x < 8 * NH) {
    float m = -INFINITY, s = 0.f;
#pragma unroll
    for (int w = 0; w < kExWarps; ++w) {
      const float2 v = red[w][threadIdx.x];
      const float nm = fmaxf(m, v.x);
      if (nm > -INFINITY) { s = s * __expf(m - nm) + v.y * __expf(v.x - nm); m = nm; }
    }
    p.part[((int64_t)b * p.Hq + h * p.G + threadIdx.x) * p.max_groups + chunk] = make_float2(m, s);
  }
}

// Plain fp32 arithmetic for any element type: one warp per page, a lane owns four dims.
// ENV: instead of the exact log-mass, the min/max envelope score (the bound Quest ranks by, Lemma 2 of the paper):
//   e_j(q) = sum_c max(q_c u_c, q_c l_c) / sqrt(d),  u_c / l_c = largest / smallest key entry of the page in dim c.
template <typename T, bool ENV>
__global__ void __launch_bounds__(kExWarps * 32) exact_generic_kernel(ExactParams p) {
  __shared__ float2 red[kExWarps][16];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  pdl_wait();
  const int Tn = p.seq_lens[b];
  const int P = (Tn + LOCKS_B - 1) / LOCKS_B;
  const int lo = chunk * kExPagesPerCta, hi = min(lo + kExPagesPerCta, P);
  const T *K = reinterpret_cast<const T *>(p.k), *Q = reinterpret_cast<const T *>(p.q);
  for (int g = 0; g < p.G; ++g) {
    float qv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) qv[u] = ldf<T>(Q, ((int64_t)b * p.Hq + h * p.G + g) * LOCKS_D + lane * 4 + u);
    float pm = -INFINITY, ps = 0.f;
    for (int page = lo + warp; page < hi; page += kExWarps) {
      const int block = p.block_table[(int64_t)b * p.Pmax + page];
      if (block < 0 || block >= p.num_blocks) {
        if (lane == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
        continue;
      }
      const int ntok = min(LOCKS_B, Tn - page * LOCKS_B);
      const int64_t base = (int64_t)block * p.sb + (int64_t)h * p.sh;
      float v;
      if (ENV) {
        float hi[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY}, lo[4] = {INFINITY, INFINITY, INFINITY, INFINITY};
        for (int i = 0; i < ntok; ++i)
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float kk = ldf<T>(K, base + (int64_t)i * p.st + lane * 4 + u);
            hi[u] = fmaxf(hi[u], kk); lo[u] = fminf(lo[u], kk);
          }
        float e = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) e += fmaxf(qv[u] * hi[u], qv[u] * lo[u]);
        v = warp_sum(e) * p.sm_scale;
      } else {
        float m = -INFINITY, s = 0.f;
        for (int i = 0; i < ntok; ++i) {
          float d = 0.f;
#pragma unroll
          for (int u = 0; u < 4; ++u) d += qv[u] * ldf<T>(K, base + (int64_t)i * p.st + lane * 4 + u);
          lse_push(m, s, warp_sum(d) * p.sm_scale);
        }
        v = m + logf(s);
      }
      if (lane == 0) {
        p.shat[((int64_t)b * p.Hq + h * p.G + g) * p.Pmax + page] = v;
        if (page >= 1 && page <= P - 2) lse_push(pm, ps, v);
      }
    }
    if (lane == 0) red[warp][g] = make_float2(pm, ps);
  }
  __syncthreads();
  if (threadIdx.x < p.G) {
    float m = -INFINITY, s = 0.f;
    for (int w = 0; w < kExWarps; ++w) {
      const float2 v = red[w][threadIdx.x];
      const float nm = fmaxf(m, v.x);
      if (nm > -INFINITY) { s = s * __expf(m - nm) + v.y * __expf(v.x - nm); m = nm; }
    }
    p.part[((int64_t)b * p.Hq + h * p.G + threadIdx.x) * p.max_groups + chunk] = make_float2(m, s);
  }
}

struct QualityParams {
  const float *mass;          // [batch][Hq][Pmax] exact page log-masses, pages 0..P-1
  const int32_t *seq_lens;
  const int32_t *ids_a, *cnt_a, *ids_r, *cnt_r;   // [batch][Hkv][k], [batch][Hkv]
  const int32_t *marked;      // [batch][n_marked] logical pages (-1: none) or nullptr
  float *out;                 // [batch][Hkv][4]: gamma, gamma_c, recall, needle
  int batch, Hq, Hkv, G, Pmax, k, n_marked;
};

__global__ void __launch_bounds__(128) quality_kernel(QualityParams p) {
  __shared__ float sh_m[4], sh_s[4];
  __shared__ float sh_acc[3];
  __shared__ int sh_cnt[4];
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t prob = (int64_t)b * p.Hkv + h;
  const int T = p.seq_lens[b], P = (T + LOCKS_B - 1) / LOCKS_B;
  const int ca = min(max(p.cnt_a[prob], 0), p.k), cr = min(max(p.cnt_r[prob], 0), p.k);
  const int32_t *A = p.ids_a + prob * p.k, *R = p.ids_r + prob * p.k;
  if (tid < 3) sh_acc[tid] = 0.f;
  if (tid < 4) sh_cnt[tid] = 0;
  __syncthreads();
  for (int g = 0; g < p.G; ++g) {
    const float *s = p.mass + ((int64_t)b * p.Hq + h * p.G + g) * p.Pmax;
    // log Z over every page of the sequence
    float m = -INFINITY, z = 0.f;
    for (int j = tid; j < P; j += 128) lse_push(m, z, s[j]);
    float M = warp_max(m);
    z = warp_sum(M > -INFINITY ? z * __expf(m - M) : 0.f);
    if (lane == 0) { sh_m[warp] = M; sh_s[warp] = z; }
    __syncthreads();
    M = fmaxf(fmaxf(sh_m[0], sh_m[1]), fmaxf(sh_m[2], sh_m[3]));
    float Z = 0.f;
    for (int w = 0; w < 4; ++w) Z += sh_m[w] > -INFINITY ? sh_s[w] * __expf(sh_m[w] - M) : 0.f;
    __syncthreads();
    // share of the pages in A
    float kept = 0.f;
    for (int j = tid; j < ca; j += 128) { const int pg = A[j]; if (pg >= 0 && pg < P) kept += __expf(s[pg] - M); }
    kept = warp_sum(kept);
    if (lane == 0) sh_s[warp] = kept;
    __syncthreads();
    if (tid == 0) {
      const float kz = (sh_s[0] + sh_s[1]) + (sh_s[2] + sh_s[3]);
      const float always = __expf(s[0] - M) + (P > 1 ? __expf(s[P - 1] - M) : 0.f);
      sh_acc[0] += kz / Z;
      sh_acc[1] += (Z - always) > 0.f ? fmaxf(kz - always, 0.f) / (Z - always) : 1.f;
    }
    __syncthreads();
  }
  // recall over candidate pages (both lists ascending; a linear probe per element is plenty here)
  int hit = 0, tot = 0, nk = 0, nh = 0;
  for (int j = tid; j < cr; j += 128) {
    const int pg = R[j];
    if (pg <= 0 || pg >= P - 1) continue;
    ++tot;
    for (int i = 0; i < ca; ++i) if (A[i] == pg) { ++hit; break; }
  }
  if (p.marked) {
    for (int j = tid; j < p.n_marked; j += 128) {
      const int pg = p.marked[(int64_t)b * p.n_marked + j];
      if (pg <= 0 || pg >= P - 1) continue;
      bool in_r = false, in_a = false;
      for (int i = 0; i < cr; ++i) in_r |= R[i] == pg;
      for (int i = 0; i < ca; ++i) in_a |= A[i] == pg;
      if (in_r) { ++nk; if (in_a) ++nh; }
    }
  }
  atomicAdd(&sh_cnt[0], hit); atomicAdd(&sh_cnt[1], tot); atomicAdd(&sh_cnt[2], nh); atomicAdd(&sh_cnt[3], nk);
  __syncthreads();
  if (tid == 0) {
    float *o = p.out + prob * 4;
    o[0] = sh_acc[0] / p.G;
    o[1] = sh_acc[1] / p.G;
    o[2] = sh_cnt[1] > 0 ? (float)sh_cnt[0] / sh_cnt[1] : 1.f;
    o[3] = sh_cnt[3] > 0 ? (float)sh_cnt[2] / sh_cnt[3] : 1.f;
  }
}

}  // namespace

int locks_launch_exact_scan(locks_ctx *c, const void *q, const locks_kv *kv, int batch, float *shat, int envelope,
                            cudaStream_t st) {
  ExactParams p;
  p.q = q; p.k = kv->k; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.shat = shat; p.part = c->part; p.status = c->status;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G; p.Pmax = c->Pmax;
  p.max_groups = c->max_groups; p.num_blocks = kv->num_blocks; p.kbud = c->k; p.sm_scale = c->cfg.sm_scale;
  const int chunks = (c->Pmax + kExPagesPerCta - 1) / kExPagesPerCta;
  c->part_slots = chunks;     // one partial per (head, CTA); chunks <= max_groups since a CTA covers 64 >= 8 pages
  c->part_balanced = 0;
  c->last_partition = 0;
  dim3 grid(chunks, p.Hkv, batch);
  if (envelope) {
    if (c->cfg.kv_dtype == LOCKS_BF16) locks_launch_pdl(exact_generic_kernel<__nv_bfloat16, true>, grid, dim3(kExWarps * 32), 0, st, p);
    else locks_launch_pdl(exact_generic_kernel<float, true>, grid, dim3(kExWarps * 32), 0, st, p);
  } else if (c->cfg.kv_dtype == LOCKS_BF16) {
    if (locks_attrs_needed(LOCKS_ATTR_EXACT)) {
      cudaFuncSetAttribute(exact_bf16_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kExSmem);
      cudaFuncSetAttribute(exact_bf16_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kExSmem);
    }
    if (c->G <= 8) locks_launch_pdl(exact_bf16_kernel<1>, grid, dim3(kExWarps * 32), kExSmem, st, p);
    else locks_launch_pdl(exact_bf16_kernel<2>, grid, dim3(kExWarps * 32), kExSmem, st, p);
  } else {
    locks_launch_pdl(exact_generic_kernel<float, false>, grid, dim3(kExWarps * 32), 0, st, p);
  }
  return locks_check_launch(c);
}

int locks_launch_quality(locks_ctx *c, const float *mass, const locks_kv *kv, int batch, const int32_t *ids_a,
                         const int32_t *cnt_a, const int32_t *ids_r, const int32_t *cnt_r, const int32_t *marked,
                         int n_marked, float *out, cudaStream_t st) {
  QualityParams p;
  p.mass = mass; p.seq_lens = kv->seq_lens; p.ids_a = ids_a; p.cnt_a = cnt_a; p.ids_r = ids_r; p.cnt_r = cnt_r;
  p.marked = n_marked > 0 ? marked : nullptr; p.out = out;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G; p.Pmax = c->Pmax; p.k = c->k;
  p.n_marked = n_marked;
  quality_kernel<<<dim3(p.Hkv, batch), 128, 0, st>>>(p);
  return locks_check_launch(c);
}
