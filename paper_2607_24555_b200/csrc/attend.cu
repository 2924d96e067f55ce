// Stage B: sparse paged attention over the selected pages (Sec. 3 "Decode-time attention", App. E):
//   o_g = sum_i softmax_i(q_g . k_i / sqrt(d)) v_i   over tokens i < T of the pages in the table,
// computed split-K: every CTA takes a slice of the page list, every warp streams whole pages
// (K tile 16x128 + V tile 16x128) through its own two-stage shared-memory ring with 16-byte async
// copies into an XOR-swizzled layout, scores them with m16n8k16 bf16 MMAs (the G query heads of the
// KV head are the M rows), keeps a running (max, sum, O) per head, and the CTA merges its warps by
// log-sum-exp.  Partial (o, lse) per split are merged by a second small kernel.
// A NULL page table means "all pages": the same kernel is the dense flash-decode baseline.
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
  float sm_scale;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

constexpr int kTile = LOCKS_B * LOCKS_D * 2;                 // 4096 B: one K or V page tile in bf16
constexpr int kAttStage = 2 * kTile;                         // K + V
constexpr int kAttSmem = LOCKS_ATT_WARPS * 2 * kAttStage;    // two stages per warp

// Resolve the idx-th page of this problem's list: logical page, physical block, valid tokens.
__device__ __forceinline__ bool resolve_page(const AttParams &p, int b, int64_t prob, int idx, int T, int &block,
                                             int &ntok) {
  const int page = p.ids ? p.ids[prob * p.kbud + idx] : idx;
  if (page < 0 || page >= p.Pmax) { set_status(p.status, LOCKS_ERR_BAD_BLOCK); return false; }
  block = p.block_table[(int64_t)b * p.Pmax + page];
  if (block < 0 || block >= p.num_blocks) { set_status(p.status, LOCKS_ERR_BAD_BLOCK); return false; }
  ntok = min(LOCKS_B, T - page * LOCKS_B);
  return ntok > 0;
}

template <int NH>
__global__ void __launch_bounds__(LOCKS_ATT_WARPS * 32) attend_bf16_kernel(AttParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int x = lane >> 2, t = lane & 3;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int64_t prob = (int64_t)b * p.Hkv + h;
  const int T = p.seq_lens[b];
  const int P = (T + LOCKS_B - 1) / LOCKS_B;
  const int npages = p.ids ? p.cnt[prob] : P;
  const int lo = split * p.pages_per_cta;
  const int hi = min(lo + p.pages_per_cta, npages);
  uint8_t *ring = smem + warp * 2 * kAttStage;
  const __nv_bfloat16 *K = reinterpret_cast<const __nv_bfloat16 *>(p.k);
  const __nv_bfloat16 *V = reinterpret_cast<const __nv_bfloat16 *>(p.v);

  // query fragments: rows = heads of the group
  uint32_t qa[8][4];
  {
    const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(p.q);
    const uint32_t *q0 = reinterpret_cast<const uint32_t *>(q + ((int64_t)b * p.Hq + h * p.G + x) * LOCKS_D);
    const uint32_t *q8 = reinterpret_cast<const uint32_t *>(q + ((int64_t)b * p.Hq + h * p.G + x + 8) * LOCKS_D);
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      qa[s][0] = (x < p.G) ? __ldg(q0 + 8 * s + t) : 0u;
      qa[s][2] = (x < p.G) ? __ldg(q0 + 8 * s + 4 + t) : 0u;
      qa[s][1] = (NH == 2 && x + 8 < p.G) ? __ldg(q8 + 8 * s + t) : 0u;
      qa[s][3] = (NH == 2 && x + 8 < p.G) ? __ldg(q8 + 8 * s + 4 + t) : 0u;
    }
  }
  const float c2 = p.sm_scale * kLog2e;

  float oacc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
  float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f};

  auto issue = [&](int idx, int stage) -> int {  // returns valid tokens (0: nothing loaded)
    int block = 0, ntok = 0;
    const bool okp = resolve_page(p, b, prob, idx, T, block, ntok);
    if (!okp) ntok = 0;
    uint8_t *kt = ring + stage * kAttStage, *vt = kt + kTile;
    const int64_t base = (int64_t)block * p.sb + (int64_t)h * p.sh;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = lane + 32 * i, tok = c >> 4, ch = c & 15;
      const int64_t off = base + (int64_t)tok * p.st + ch * 8;
      const int so = tok * 256 + ((ch ^ (tok & 7)) << 4);
      cp_async16(kt + so, K + off, tok < ntok);   // rows past the sequence end are zero-filled
      cp_async16(vt + so, V + off, tok < ntok);
    }
    cp_async_commit();
    return ntok;
  };

  const int first = lo + warp;
  int ntok_cur = 0, ntok_next = 0;
  if (first < hi) ntok_cur = issue(first, 0);
  int j = 0;
  for (int idx = first; idx < hi; idx += LOCKS_ATT_WARPS, ++j) {
    const int stage = j & 1;
    const bool more = idx + LOCKS_ATT_WARPS < hi;
    if (more) ntok_next = issue(idx + LOCKS_ATT_WARPS, stage ^ 1);
    if (more) cp_async_wait<1>(); else cp_async_wait<0>();
    __syncwarp();
    const uint8_t *kt = ring + stage * kAttStage, *vt = kt + kTile;
    const int ntok = ntok_cur;
    // ---- S = q K^T  (16 heads x 16 tokens)
    float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    {
      const int m = lane >> 3, rr = lane & 7;
#pragma unroll
      for (int s2 = 0; s2 < 4; ++s2) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int tok = nt * 8 + rr, ch = 4 * s2 + m;
          uint32_t r[4];
          ldsm_x4(r, kt + tok * 256 + ((ch ^ (tok & 7)) << 4));
          mma_bf16(sacc[nt], qa[2 * s2][0], qa[2 * s2][1], qa[2 * s2][2], qa[2 * s2][3], r[0], r[1]);
          mma_bf16(sacc[nt], qa[2 * s2 + 1][0], qa[2 * s2 + 1][1], qa[2 * s2 + 1][2], qa[2 * s2 + 1][3], r[2], r[3]);
        }
      }
    }
    // ---- online softmax per head row
    uint32_t pa[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      float v0 = sacc[0][2 * hh] * c2, v1 = sacc[0][2 * hh + 1] * c2;
      float v2 = sacc[1][2 * hh] * c2, v3 = sacc[1][2 * hh + 1] * c2;
      if (2 * t >= ntok) v0 = -INFINITY;
      if (2 * t + 1 >= ntok) v1 = -INFINITY;
      if (8 + 2 * t >= ntok) v2 = -INFINITY;
      if (9 + 2 * t >= ntok) v3 = -INFINITY;
      float m = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
      const float mnew = fmaxf(mrun[hh], m);
      const float msafe = (mnew == -INFINITY) ? 0.f : mnew;
      const float alpha = ex2f(mrun[hh] - msafe);
      const float p0 = ex2f(v0 - msafe), p1 = ex2f(v1 - msafe), p2 = ex2f(v2 - msafe), p3 = ex2f(v3 - msafe);
      lrun[hh] = lrun[hh] * alpha + (p0 + p1) + (p2 + p3);
      mrun[hh] = mnew;
#pragma unroll
      for (int i = 0; i < 16; ++i) { oacc[i][2 * hh] *= alpha; oacc[i][2 * hh + 1] *= alpha; }
      pa[hh] = pack_bf16(p0, p1);
      pa[2 + hh] = pack_bf16(p2, p3);
    }
    // ---- O += P V
    {
      const int m = lane >> 3, rr = lane & 7;
      const int tok = (m & 1) * 8 + rr;
#pragma unroll
      for (int ntp = 0; ntp < 8; ++ntp) {
        const int ch = 2 * ntp + (m >> 1);
        uint32_t r[4];
        ldsm_x4_trans(r, vt + tok * 256 + ((ch ^ (tok & 7)) << 4));
        mma_bf16(oacc[2 * ntp], pa[0], pa[1], pa[2], pa[3], r[0], r[1]);
        mma_bf16(oacc[2 * ntp + 1], pa[0], pa[1], pa[2], pa[3], r[2], r[3]);
      }
    }
    __syncwarp();
    ntok_cur = ntok_next;
  }
  cp_async_wait<0>();
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) {
    lrun[hh] += __shfl_xor_sync(0xffffffffu, lrun[hh], 1);
    lrun[hh] += __shfl_xor_sync(0xffffffffu, lrun[hh], 2);
  }
  __syncthreads();  // every warp is done with its ring: reuse it for the merge
  float *wo = reinterpret_cast<float *>(ring);          // [16][128] fp32
  float *wm = wo + 16 * LOCKS_D, *wl = wm + 16;          // [16], [16]
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) {
    const int row = x + 8 * hh;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
      *reinterpret_cast<float2 *>(wo + row * LOCKS_D + nt * 8 + 2 * t) = make_float2(oacc[nt][2 * hh], oacc[nt][2 * hh + 1]);
    if (t == 0) { wm[row] = mrun[hh]; wl[row] = lrun[hh]; }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < p.G * LOCKS_D; e += LOCKS_ATT_WARPS * 32) {
    const int g = e / LOCKS_D, dim = e - g * LOCKS_D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < LOCKS_ATT_WARPS; ++w)
      M = fmaxf(M, reinterpret_cast<const float *>(smem + w * 2 * kAttStage)[16 * LOCKS_D + g]);
    float L = 0.f, o = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < LOCKS_ATT_WARPS; ++w) {
        const float *ww = reinterpret_cast<const float *>(smem + w * 2 * kAttStage);
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
  if (p.splits == 1) return;
  // the last CTA of this (request, KV head) to arrive merges the splits' partials by log-sum-exp
  __shared__ int sh_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) sh_last = (atomicAdd(&p.done[prob], 1) == p.splits - 1);
  __syncthreads();
  if (!sh_last) return;
  __threadfence();
  for (int e = threadIdx.x; e < p.G * LOCKS_D; e += LOCKS_ATT_WARPS * 32) {
    const int g = e / LOCKS_D, dim = e - g * LOCKS_D;
    const int64_t row = (int64_t)b * p.Hq + h * p.G + g;
    const float *pl = p.part_lse + row * p.splits;
    float M = -INFINITY;
    for (int s2 = 0; s2 < p.splits; ++s2) M = fmaxf(M, __ldcg(pl + s2));
    float L = 0.f, acc = 0.f;
    if (M > -INFINITY) {
      for (int s2 = 0; s2 < p.splits; ++s2) {
        const float w = ex2f(__ldcg(pl + s2) - M);
        L += w;
        acc += w * __ldcg(p.part_o + (row * p.splits + s2) * LOCKS_D + dim);
      }
      acc /= L;
    }
    reinterpret_cast<__nv_bfloat16 *>(p.out)[row * LOCKS_D + dim] = __float2bfloat16_rn(acc);
    if (p.lse && dim == 0) p.lse[row] = (M > -INFINITY) ? (M + log2f(L)) * kLn2 : -INFINITY;
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
  const int64_t prob = (int64_t)b * p.Hkv + h;
  const int Tn = p.seq_lens[b];
  const int P = (Tn + LOCKS_B - 1) / LOCKS_B;
  const int npages = p.ids ? p.cnt[prob] : P;
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
    const int64_t base = (int64_t)block * p.sb + (int64_t)h * p.sh;
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

template <typename T>
__global__ void __launch_bounds__(128) attend_merge_kernel(const float *part_o, const float *part_lse, int splits,
                                                           T *out, float *lse, int Hq) {
  const int hq = blockIdx.x, b = blockIdx.y, dim = threadIdx.x;
  const int64_t row = (int64_t)b * Hq + hq;
  const float *pl = part_lse + row * splits;
  float M = -INFINITY;
  for (int s = 0; s < splits; ++s) M = fmaxf(M, pl[s]);
  float L = 0.f, acc = 0.f;
  if (M > -INFINITY) {
    for (int s = 0; s < splits; ++s) {
      const float w = exp2f(pl[s] - M);
      L += w;
      acc += w * part_o[(row * splits + s) * LOCKS_D + dim];
    }
    acc /= L;
  }
  stf<T>(out, row * LOCKS_D + dim, acc);
  if (lse && dim == 0) lse[row] = (M > -INFINITY) ? (M + log2f(L)) * kLn2 : -INFINITY;
}

}  // namespace

int locks_launch_attend(locks_ctx *c, const void *q, const locks_kv *kv, int batch, const int32_t *ids,
                        const int32_t *cnt, void *out, float *lse, cudaStream_t st) {
  AttParams p;
  p.q = q; p.k = kv->k; p.v = kv->v; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.ids = ids; p.cnt = cnt;
  p.part_o = c->att_o; p.part_lse = c->att_lse; p.out = out; p.lse = lse; p.status = c->status;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G; p.Pmax = c->Pmax;
  p.kbud = c->k; p.num_blocks = kv->num_blocks; p.sm_scale = c->cfg.sm_scale;
  const bool dense = ids == nullptr;
  // one wave: as many splits per problem as resident CTA slots allow, at least one page per warp
  const int npages = dense ? c->Pmax : c->k;
  const int slots = c->num_sms * LOCKS_ATT_CTAS_PER_SM;
  int splits = slots / (batch * p.Hkv);
  const int most = (npages + LOCKS_ATT_WARPS - 1) / LOCKS_ATT_WARPS;
  if (splits > most) splits = most;
  if (splits > LOCKS_ATT_MAX_SPLITS) splits = LOCKS_ATT_MAX_SPLITS;
  if (splits < 1) splits = 1;
  p.pages_per_cta = (npages + splits - 1) / splits;
  p.splits = (npages + p.pages_per_cta - 1) / p.pages_per_cta;
  p.done = c->att_done;
  const bool bf = c->cfg.kv_dtype == LOCKS_BF16;
  if (bf) {
    static bool attr_done = false;
    if (!attr_done) {
      cudaFuncSetAttribute(attend_bf16_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
      cudaFuncSetAttribute(attend_bf16_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem);
      attr_done = true;
    }
    dim3 grid(p.splits, p.Hkv, batch);
    if (c->G <= 8) attend_bf16_kernel<1><<<grid, LOCKS_ATT_WARPS * 32, kAttSmem, st>>>(p);
    else attend_bf16_kernel<2><<<grid, LOCKS_ATT_WARPS * 32, kAttSmem, st>>>(p);
  } else {
    dim3 grid(p.splits, p.Hq, batch);
    attend_generic_kernel<float><<<grid, 128, 0, st>>>(p);
  }
  int rc = locks_check_launch(c);
  if (rc != LOCKS_OK || p.splits == 1 || bf) return rc;   // the bf16 kernel merges its own splits
  dim3 mg(p.Hq, batch);
  attend_merge_kernel<float><<<mg, 128, 0, st>>>(c->att_o, c->att_lse, p.splits, reinterpret_cast<float *>(out), lse,
                                                 p.Hq);
  return locks_check_launch(c);
}
