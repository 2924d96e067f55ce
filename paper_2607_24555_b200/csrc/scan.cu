// Stage A, part 1: scan every resident page summary and score it (Eq. 1 of the paper):
//   s^_j(q_g) = log sum_{i in P_j} exp[(q_g . mu_j + (V_j^T q_g) . c_i) / sqrt(d)]
// for every page j <= P-2 of every request and every query head g, plus a per-(head, 8-page group)
// partial (max, sum exp) over the candidate pages 1..P-2 that the selector turns into log Z_g.
//
// Two kernels:
//   scan_generic_kernel   any format / rank / dtype, plain fp32 ALU arithmetic (parity config, fallback
//                         shapes).  One warp per group of 8 pages.
//   scan_i4_kernel<R>     the bytes-bound path for int4/int8 blobs of rank R = 2, 4, 8 with bf16 queries (ranks
//                         below 8 run the rank-8 tile with the missing ranks fed as zeros).  Persistent warps,
//                         each streaming groups of 8 blobs through its own shared-memory ring with bulk
//                         async copies (TMA engine) and mbarriers, no CTA-wide synchronisation.  Per page pair:
//                           MMA#1  P[2 pages x 8 ranks, heads] = codesV[16 x d] . q^T[d x heads]   (8 x m16n8k16 fp16)
//                         per page, after an 8x8 movmatrix transpose of the fp16 hi/lo projection:
//                           MMA#2  L[heads, tokens] = (P_hi | P_lo)[heads x 16] . codesC^T          (2 x m16n8k16 fp16)
//                         and per 8 pages the centroid dots a[heads, pages] (8 x m16n8k16 fp16).
#include <cstring>
#include <cuda.h>            // CUtensorMap (types only; the encoder is fetched from the driver at run time)
#include <cudaTypedefs.h>
#include "locks_internal.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct ScanParams {
  const void *q;
  const uint8_t *summ;
  const int32_t *block_table;
  const int32_t *seq_lens;
  float *shat;
  float2 *part;
  int32_t *part_cnt;   // [batch][Hkv] partials written per head of a problem (balanced partition)
  int32_t *status;
  int batch, Hq, Hkv, G, Pmax, max_groups, num_blocks, k, S, r;
  int B;   // tokens per page
  float sm_scale;
  // decode step with an appended token: lengths count the token that the selector's kernel is about to
  // write (seq_inc = 1); the first CTA publishes them, and the append position, for the step's later kernels
  int cta_reduce;     // every warp of a CTA works on one problem only: one partial per (head, CTA)
  int wpp, nslots;    // strided partition: warps per problem, problems in flight
  int use_gather;     // stage four summaries per tensor-map gather instead of one bulk copy each
  int seq_inc;
  int scorer;         // generic kernel only: LOCKS_SCORER_* (the summary's own score, or a rival functional of it)
  int32_t *seq_eff;   // [2][max_batch]: effective length, append position (-1: none) -- or nullptr
};

// Length of request b as this step sees it.  A sequence that has no room for the token keeps its length.
__device__ __forceinline__ int step_len(const ScanParams &p, int b) {
  return min(p.seq_lens[b] + p.seq_inc, p.Pmax * p.B);
}

__device__ __forceinline__ void publish_lengths(const ScanParams &p, bool first_cta, int tid, int nthreads) {
  if (!first_cta || !p.seq_eff) return;
  for (int b = tid; b < p.batch; b += nthreads) {
    const int T0 = p.seq_lens[b], T1 = T0 + p.seq_inc;
    const bool room = T1 <= p.Pmax * p.B;
    if (!room) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
    p.seq_eff[b] = room ? T1 : T0;
    p.seq_eff[p.batch + b] = (room && p.seq_inc) ? T0 : -1;
  }
}

// ------------------------------------------------------------------------------------------------
// generic path
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ float i4_basis_val(const uint8_t *blob, int l, int c) {
  int t = c >> 5, w = c & 31, s = w >> 2, half = (w >> 1) & 1, e = w & 1;
  int j = s >> 1, i = ((s & 1) << 1) | half, nib = i + 4 * e;
  int byte = (l * 4 + t) * 16 + j * 4 + (nib >> 1);
  return (float)(((blob[byte] >> ((nib & 1) * 4)) & 15) - 8);
}
__device__ __forceinline__ float i4_mu_val(const uint8_t *blob, int r, int c, int B) {
  int t = c >> 5, w = c & 31, s = w >> 2, half = (w >> 1) & 1, e = w & 1;
  return (float)((int)blob[i4_off_mu(r, B) + t * 32 + s * 4 + e * 2 + half] - 128);
}
// coefficients and their scales: interleaved for the tensor-core fragments at B = 16, row-major (token, rank) otherwise
__device__ __forceinline__ float i4_coef_val(const uint8_t *blob, int r, int i, int l, int B) {
  int x = i & 7, hi = i >> 3, tp = l >> 1, e = l & 1;
  const int pos = B == LOCKS_B ? (x * (r / 2) + tp) * 4 + hi * 2 + e : i * r + l;
  return (float)((int)blob[i4_off_coef(r) + pos] - 128);
}
__device__ __forceinline__ float i4_sc_val(const uint8_t *blob, int r, int i, int B) {
  int t = (i & 7) >> 1, e = i & 1, hi = i >> 3;
  const int pos = B == LOCKS_B ? t * 4 + hi * 2 + e : i;
  return __half2float(*reinterpret_cast<const __half *>(blob + i4_off_sc(r, B) + 2 * pos));
}

template <int FMT, typename QT>
__global__ void __launch_bounds__(128) scan_generic_kernel(ScanParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = blockIdx.x * 4 + warp, h = blockIdx.y, b = blockIdx.z;
  pdl_wait();
  publish_lengths(p, (blockIdx.x | blockIdx.y | blockIdx.z) == 0, threadIdx.x, 128);
  const int T = step_len(p, b);
  const int B = p.B;                  // 16, 32 or 64 tokens per page: lane i holds tokens i and i + 32
  const int P = (T + B - 1) / B;
  if (P <= p.k) return;               // every page is kept: nothing to rank
  const int nsc = P - 1;              // pages 0 .. P-2 are scored
  if (grp * LOCKS_GROUP >= nsc) return;
  const int r = p.r;
  const QT *q = reinterpret_cast<const QT *>(p.q);
  for (int g = 0; g < p.G; ++g) {
    const int hq = h * p.G + g;
    float qv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) qv[u] = ldf<QT>(q, ((int64_t)b * p.Hq + hq) * LOCKS_D + lane * 4 + u);
    float pm = -INFINITY, ps = 0.f;
    for (int pi = 0; pi < LOCKS_GROUP; ++pi) {
      const int page = grp * LOCKS_GROUP + pi;
      if (page >= nsc) break;
      int block = p.block_table[(int64_t)b * p.Pmax + page];
      if (block < 0 || block >= p.num_blocks) {
        if (lane == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
        continue;
      }
      const uint8_t *blob = p.summ + ((int64_t)block * p.Hkv + h) * p.S;
      float proj[16];
      float a = 0.f;
      if (FMT == LOCKS_FMT_F32) {
        const float *f = reinterpret_cast<const float *>(blob);
#pragma unroll
        for (int u = 0; u < 4; ++u) a += f[lane * 4 + u] * qv[u];
        for (int l = 0; l < r; ++l) {
          float s = 0.f;
#pragma unroll
          for (int u = 0; u < 4; ++u) s += f[LOCKS_D + l * LOCKS_D + lane * 4 + u] * qv[u];
          proj[l] = warp_sum(s);
        }
      } else if (FMT == LOCKS_FMT_I8 || FMT == LOCKS_FMT_BF16) {
        constexpr int W = FMT == LOCKS_FMT_BF16 ? 2 : 1;
        const float smu = __half2float(*reinterpret_cast<const __half *>(blob + wb_off_smu(r, W, B)));
#pragma unroll
        for (int u = 0; u < 4; ++u) a += (float)((int)blob[wb_off_mu(r, W, B) + lane * 4 + u] - 128) * qv[u];
        a *= smu;
        for (int l = 0; l < r; ++l) {
          float s = 0.f;
          if (FMT == LOCKS_FMT_I8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) s += (float)((int)blob[l * LOCKS_D + lane * 4 + u] - 128) * qv[u];
            s *= __half2float(*reinterpret_cast<const __half *>(blob + wb_off_sv(r, W, B) + 2 * l));
          } else {
#pragma unroll
            for (int u = 0; u < 4; ++u)
              s += __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(blob)[l * LOCKS_D + lane * 4 + u]) * qv[u];
          }
          proj[l] = warp_sum(s);
        }
      } else {
        const float smu = __half2float(*reinterpret_cast<const __half *>(blob + i4_off_smu(r, B)));
#pragma unroll
        for (int u = 0; u < 4; ++u) a += i4_mu_val(blob, r, lane * 4 + u, B) * qv[u];
        a *= smu;
        for (int l = 0; l < r; ++l) {
          float s = 0.f;
#pragma unroll
          for (int u = 0; u < 4; ++u) s += i4_basis_val(blob, l, lane * 4 + u) * qv[u];
          const float sv = __half2float(*reinterpret_cast<const __half *>(blob + i4_off_sv(r, B) + 2 * l));
          proj[l] = warp_sum(s) * sv;
        }
      }
      a = warp_sum(a);
      float logit[2] = {-INFINITY, -INFINITY};   // tokens lane and lane + 32
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int tok = lane + 32 * half;
        if (tok >= B) continue;
        float s = 0.f;
        if (FMT == LOCKS_FMT_F32) {
          const float *f = reinterpret_cast<const float *>(blob) + LOCKS_D + r * LOCKS_D + tok * r;
          for (int l = 0; l < r; ++l) s += proj[l] * f[l];
        } else if (FMT == LOCKS_FMT_I8 || FMT == LOCKS_FMT_BF16) {
          constexpr int W = FMT == LOCKS_FMT_BF16 ? 2 : 1;
          for (int l = 0; l < r; ++l) s += proj[l] * (float)((int)blob[wb_off_coef(r, W) + tok * r + l] - 128);
          s *= __half2float(*reinterpret_cast<const __half *>(blob + wb_off_sc(r, W, B) + 2 * tok));
        } else {
          for (int l = 0; l < r; ++l) s += proj[l] * i4_coef_val(blob, r, tok, l, B);
          s *= i4_sc_val(blob, r, tok, B);
        }
        logit[half] = p.sm_scale * (a + s);
      }
      float sh;
      if (p.scorer == LOCKS_SCORER_CENTROID) {          // the centroid term alone: q.mu / sqrt(d) + log B
        sh = p.sm_scale * a + logf((float)B);
      } else if (p.scorer == LOCKS_SCORER_MOMENT) {     // second-cumulant truncation of the mass (moment core)
        float z2 = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half)
          if (lane + 32 * half < B) { const float zi = logit[half] - p.sm_scale * a; z2 = fmaf(zi, zi, z2); }
        sh = p.sm_scale * a + logf((float)B) + warp_sum(z2) * (0.5f / B);
      } else {
        const float mx = warp_max(fmaxf(logit[0], logit[1]));
        float e = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half)
          if (lane + 32 * half < B) e += expf(logit[half] - mx);
        sh = mx + logf(warp_sum(e));
      }
      if (lane == 0) {
        p.shat[((int64_t)b * p.Hq + hq) * p.Pmax + page] = sh;
        if (page >= 1) {  // candidates only
          const float nm = fmaxf(pm, sh);
          ps = ps * expf(pm - nm) + expf(sh - nm);
          pm = nm;
        }
      }
    }
    if (lane == 0) p.part[((int64_t)b * p.Hq + hq) * p.max_groups + grp] = make_float2(pm, ps);
  }
}

// ------------------------------------------------------------------------------------------------
// r8i4 tensor path
// ------------------------------------------------------------------------------------------------

constexpr int kScanWarps = 8;
constexpr int kScanStages = 2;
constexpr int kScanCtasPerSm = 2;
constexpr int kStageBytes = LOCKS_GROUP * i4_stride(8);   // 6656: a stage holds 8 summaries of any rank
constexpr int kScanRedBytes = kScanWarps * 16 * 8;         // (max, sum) of 16 heads per warp, for the CTA-level merge
constexpr int kScanSmem = kScanWarps * (kScanStages * kStageBytes + 64) + kScanRedBytes;
constexpr bool kScanBulk = LOCKS_SCAN_BULK;             // true: cp.async.bulk + mbarrier, false: 16-byte cp.async

// (a & b) | c in one LOP3 with both constants held in registers
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t f16x2_sub(uint32_t v, uint32_t c) {
  __half2 r = __hsub2(*reinterpret_cast<__half2 *>(&v), *reinterpret_cast<__half2 *>(&c));
  return *reinterpret_cast<uint32_t *>(&r);
}
__device__ __forceinline__ uint32_t f16x2_fma(uint32_t a, uint32_t b, uint32_t c) {
  __half2 r = __hfma2(*reinterpret_cast<__half2 *>(&a), *reinterpret_cast<__half2 *>(&b), *reinterpret_cast<__half2 *>(&c));
  return *reinterpret_cast<uint32_t *>(&r);
}
__device__ __forceinline__ float2 h2f2(uint32_t v) { return __half22float2(*reinterpret_cast<__half2 *>(&v)); }
__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fast_lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// D = A * B with a zero accumulator (no register is spent on the zeros)
__device__ __forceinline__ void mma_f16_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%10,%10,%10,%10};\n"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

struct Cursor {
  int prob, grp, nsc, b, h;   // (request, KV head) of prob are refreshed only when prob changes
  const int32_t *bt;          // block-table row of request b
};

// Four rows of a 2D tensor map (box = one row) to consecutive rows in shared memory, completion on an mbarrier.
__device__ __forceinline__ void tma_gather4(void *dst, const CUtensorMap *tmap, int r0, int r1, int r2, int r3,
                                            uint64_t *bar, uint64_t pol) {
  if (LOCKS_SCAN_HINT_LOAD)
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes.L2::cache_hint [%0], "
        "[%1, {%2, %3, %4, %5, %6}], [%7], %8;\n" ::"r"(smem_u32(dst)),
        "l"(tmap), "r"(0), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(smem_u32(bar)), "l"(pol)
        : "memory");
  else
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, "
        "%5, %6}], [%7];\n" ::"r"(smem_u32(dst)),
        "l"(tmap), "r"(0), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ uint32_t movm_trans(uint32_t v) {
  uint32_t d;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(v));
  return d;
}

// NH = number of 8-head column tiles of the query in use (1: G <= 8, 2: G <= 16).
//
// Numerics.  Every stored code enters the tensor core exactly.
//  * A basis nibble n = code + 8 masked in place is an fp16 SUBNORMAL: at bits 0-3 it reads
//    n 2^-24, at bits 4-7 it reads 16 n 2^-24 (both below 1024, so the encoding is linear); the
//    factor 16 is undone exactly by holding the matching query elements divided by 16, the common
//    2^-24 by an exact power-of-two multiply of the fp32 accumulator, and the +8 offset by
//    subtracting 8 sum_c q'[c] (one fp32 constant per head).
//  * Coefficient and centroid bytes u = code + 128 are placed in the mantissa of 0x6400 (1024 + u)
//    and the 1152 is subtracted in fp16, which is exact.
//  * The query row is scaled by a power of two so that max|q| < 0.5 and converted to fp16 (bf16's
//    8 significant bits fit; only elements below 2^-14 of the row maximum can round, by at most
//    2^-25 of it).  Products are exact, sums are fp32; the projection is carried into the second
//    MMA as an fp16 hi + lo pair (22 significant bits).
// PK (G <= 4 only): the 8 head columns hold the group twice, so that after MMA#1 the projection, MMA#2 and
// the log-sum-exp handle two pages at once (rows 0-3 = page A's heads, rows 4-7 = page B's heads, the two
// pages separated along K) instead of leaving half of the lanes idle.
template <int R, int NH, bool PK, bool CR, bool BAL>
__global__ void __launch_bounds__(kScanWarps * 32, kScanCtasPerSm) scan_i4_kernel(ScanParams p, const __grid_constant__ CUtensorMap tmap) {
  constexpr int kBlob = i4_stride(R);   // stored bytes of one summary; a stage keeps room for rank-8 blobs
  // Summaries 4-7 of a stage start on a 128-byte boundary (the destination of the second tensor-map gather):
  // 4 x 832 bytes already is one, 4 x 336 and 4 x 496 need 64 bytes of padding
  constexpr int kHalfPad = (4 * kBlob) % 128 ? 128 - (4 * kBlob) % 128 : 0;
  auto boff = [](int pg) { return pg * kBlob + (kHalfPad ? (pg >> 2) * kHalfPad : 0); };   // offset of summary pg in a stage
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int x = lane >> 2, t = lane & 3;
  uint8_t *ring = smem + warp * (kScanStages * kStageBytes);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kScanWarps * kScanStages * kStageBytes + warp * 64);
  if (lane == 0) {
    for (int s = 0; s < kScanStages; ++s) mbar_init(&full[s], 1);
    fence_barrier_init();
  }
  __syncwarp();
  pdl_trigger();   // single-wave kernel: the selector may be scheduled as SMs drain
  pdl_wait();      // sequence lengths and the previous consumers of the workspace are done
  publish_lengths(p, blockIdx.x == 0, threadIdx.x, kScanWarps * 32);

  // Two partitions of the (problem, 8-page group) units over the warps, chosen per launch by the host.
  // Strided (BAL = false): `wpp` warps share a problem and stride its groups (slot = problem, sub = position
  // among its warps); best when the sequences are about equally long.  Balanced (BAL = true): every warp owns
  // an equally long contiguous range of units, whatever the mix of sequence lengths, at the price of a few
  // hundred instructions of set-up per warp.
  static_assert(!(CR && BAL), "the CTA-level merge needs the strided partition");
  const int W = gridDim.x * kScanWarps;
  const int wid = blockIdx.x * kScanWarps + warp;
  const int nprob = p.batch * p.Hkv;
  const int wpp = p.wpp, nslots = p.nslots;
  const int slot = wid / wpp, sub = wid - slot * wpp;
  if (!BAL && slot >= nslots) return;
  const int gstep = BAL ? 1 : wpp, pstep = BAL ? 1 : nslots, g0 = BAL ? 0 : sub;   // cursor stepping

  auto groups_of = [&](int b) {   // 8-page groups of scored pages of request b
    const int P = (step_len(p, b) + LOCKS_B - 1) / LOCKS_B;
    return P <= p.k ? 0 : (P - 1 + LOCKS_GROUP - 1) / LOCKS_GROUP;
  };
  int n_units = 0x7fffffff;   // balanced: units this warp owns
  int pslot_first = 0;        // balanced: partial slot of the first problem this warp touches
  Cursor cp{slot, sub, 0, 0, 0, p.block_table};
  if (BAL) {
    auto scan32 = [&](int v) {   // inclusive prefix sum over the lanes
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += up;
      }
      return v;
    };
    // groups per request, 32 requests at a time; the first chunk's totals are kept for the search below
    const int ng0 = lane < p.batch ? groups_of(lane) : 0;
    const int incl0 = scan32(ng0);
    int tot = __shfl_sync(0xffffffffu, incl0, 31);
    if (p.batch > 32) {
      int more = 0;
      for (int b = 32 + lane; b < p.batch; b += 32) more += groups_of(b);
#pragma unroll
      for (int o = 16; o; o >>= 1) more += __shfl_xor_sync(0xffffffffu, more, o);
      tot += more;
    }
    // U = q Weff + rem units over the first Weff = min(W, U) warps: the first rem warps own q + 1, the others q
    const int U = tot * p.Hkv, Weff = min(W, U);
    if (wid >= Weff) return;
    const int uq = U / Weff, urem = U - uq * Weff;
    const int u0 = wid * uq + min(wid, urem);
    n_units = uq + (wid < urem ? 1 : 0);
    // the request that holds unit u0 (a request holds Hkv * groups consecutive units)
    int base = 0, fb = 0, fstart = 0, fng = 1;
    for (int b0 = 0; b0 < p.batch; b0 += 32) {
      const int ng = b0 == 0 ? ng0 : ((b0 + lane < p.batch) ? groups_of(b0 + lane) : 0);
      const int incl = (b0 == 0 ? incl0 : scan32(ng)) * p.Hkv;
      const int chunk_total = __shfl_sync(0xffffffffu, incl, 31);
      if (u0 < base + chunk_total) {
        const int l = __ffs(__ballot_sync(0xffffffffu, base + incl > u0)) - 1;
        fb = b0 + l;
        fng = __shfl_sync(0xffffffffu, ng, l);
        fstart = base + __shfl_sync(0xffffffffu, incl, l) - fng * p.Hkv;
        break;
      }
      base += chunk_total;
    }
    const int r = u0 - fstart, hh0 = r / fng;
    cp.prob = fb * p.Hkv + hh0;
    cp.grp = r - hh0 * fng;
    // partials of a problem sit at (warp - first warp that owns one of its units): 0 for every problem this
    // warp enters at its first group; for the first one, count the warps between its first unit and u0
    if (cp.grp > 0) {
      const int us = u0 - cp.grp, big = urem * (uq + 1);
      const int wf = us < big ? us / (uq + 1) : urem + (us - big) / uq;
      pslot_first = wid - wf;
    }
  }

  // the summaries stream through L2 once; the scores are what the selector reads next
  const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
  auto store_score = [&](float *dst, float v) {
    if (LOCKS_SCAN_HINT_STORE) st_f32_hint(dst, v, pol_keep);
    else *dst = v;
  };
  auto enter = [&](Cursor &c) {   // refresh the per-problem fields of the cursor
    c.b = c.prob / p.Hkv;
    c.h = c.prob - c.b * p.Hkv;
    const int T = step_len(p, c.b);
    const int P = (T + LOCKS_B - 1) / LOCKS_B;
    c.nsc = (P <= p.k) ? 0 : P - 1;
    c.bt = p.block_table + (int64_t)c.b * p.Pmax;
  };
  auto settle = [&](Cursor &c) {  // move to the next non-empty position at or after (prob, grp)
    while (c.prob < nprob && c.grp * LOCKS_GROUP >= c.nsc) {
      c.prob += pstep;
      c.grp = g0;
      if (c.prob < nprob) enter(c);
    }
  };
  // `more`: the warp owns units past this one (balanced partition; the strided one ends at the last problem)
  auto advance = [&](Cursor &c, bool more) {
    c.grp += gstep;
    if (BAL && !more) c.prob = nprob;
    else settle(c);
  };
  // the physical block of page (grp*8 + lane) of the producer cursor, fetched one group ahead of use
  auto fetch_block = [&](const Cursor &c) -> int {
    if (c.prob >= nprob) return 0;
    const int page = c.grp * LOCKS_GROUP + lane;
    if (lane >= LOCKS_GROUP || page >= c.nsc) return 0;
    return c.bt[page];
  };
  auto issue = [&](int stage, const Cursor &c, int block) {
    const int h = c.h;
    const int nvalid = min(LOCKS_GROUP, c.nsc - c.grp * LOCKS_GROUP);
    if (lane < nvalid && (block < 0 || block >= p.num_blocks)) {
      set_status(p.status, LOCKS_ERR_BAD_BLOCK);
      block = 0;
    }
    if (p.use_gather) {
      // Summaries are rows of a 2D tensor [block * Hkv + head][S bytes]: one gather fetches four of them, so a
      // group costs two copy instructions instead of eight (about 3 of 115 instructions per summary; the
      // staging throughput itself does not change).  Slots past the last page repeat the group's first row.
      int row = block * p.Hkv + h;
      row = __shfl_sync(0xffffffffu, row, lane < nvalid ? lane : 0);
      const int r1 = __shfl_sync(0xffffffffu, row, 1), r2 = __shfl_sync(0xffffffffu, row, 2);
      const int r3 = __shfl_sync(0xffffffffu, row, 3), r4 = __shfl_sync(0xffffffffu, row, 4);
      const int r5 = __shfl_sync(0xffffffffu, row, 5), r6 = __shfl_sync(0xffffffffu, row, 6);
      const int r7 = __shfl_sync(0xffffffffu, row, 7);
      if (lane == 0) {
        uint8_t *dst = ring + stage * kStageBytes;
        mbar_expect_tx(&full[stage], (uint32_t)(nvalid > 4 ? 8 : 4) * kBlob);
        tma_gather4(dst, &tmap, row, r1, r2, r3, &full[stage], pol_stream);
        if (nvalid > 4) tma_gather4(dst + boff(4), &tmap, r4, r5, r6, r7, &full[stage], pol_stream);
      }
    } else if (kScanBulk) {
      if (lane == 0) mbar_expect_tx(&full[stage], (uint32_t)nvalid * kBlob);
      __syncwarp();
      if (lane < nvalid) {
        if (LOCKS_SCAN_HINT_LOAD)
          bulk_g2s_hint(ring + stage * kStageBytes + boff(lane), p.summ + ((int64_t)block * p.Hkv + h) * kBlob, kBlob,
                        &full[stage], pol_stream);
        else
          bulk_g2s(ring + stage * kStageBytes + boff(lane), p.summ + ((int64_t)block * p.Hkv + h) * kBlob, kBlob,
                   &full[stage]);
      }
    } else {
      // 16-byte chunks of a blob are dealt to the lanes
      uint8_t *dst = ring + stage * kStageBytes;
#pragma unroll
      for (int pg = 0; pg < LOCKS_GROUP; ++pg) {
        const int blk = __shfl_sync(0xffffffffu, block, pg);
        const uint8_t *src = p.summ + ((int64_t)blk * p.Hkv + h) * kBlob;
        if (pg < nvalid)
          for (int c = lane; c < kBlob / 16; c += 32) cp_async16(dst + boff(pg) + c * 16, src + c * 16, true);
      }
      cp_async_commit();
    }
  };

  Cursor cc;
  // strided partition: the first group's position does not depend on the lengths, so its block ids are fetched
  // beside the length instead of after it (block-table slots past a sequence's pages are readable, just unused)
  int spec_block = 0;
  if (!BAL && slot < nprob && lane < LOCKS_GROUP && sub * LOCKS_GROUP + lane < p.Pmax)
    spec_block = p.block_table[(int64_t)(slot / p.Hkv) * p.Pmax + sub * LOCKS_GROUP + lane];
  if (cp.prob < nprob) enter(cp);
  settle(cp);
  cc = cp;
  int inflight = 0;
  int next_block;
  if (!BAL && cp.prob == slot && cp.grp == sub)
    next_block = (lane < LOCKS_GROUP && sub * LOCKS_GROUP + lane < cp.nsc) ? spec_block : 0;
  else
    next_block = fetch_block(cp);
#pragma unroll
  for (int s = 0; s < kScanStages; ++s) {
    if (cp.prob < nprob) {
      issue(s, cp, next_block);
      ++inflight;
      advance(cp, inflight < n_units);
      next_block = fetch_block(cp);
    }
  }

  const uint32_t kM0 = 0x000F000Fu, kM1 = 0x00F000F0u;
  uint32_t kMB = 0x00FF00FFu, kMagic = 0x64006400u;
  asm volatile("" : "+r"(kMB), "+r"(kMagic));
  const uint32_t kSub128 = 0x64806480u;    // 1152 = 1024 + 128
  const uint32_t kSixteen = 0x4C004C00u;   // 16.0
  const uint32_t kNeg16x = 0xF480F480u;    // -18432 = -16 * 1152

  // query of the current problem: qb0/qb2 = this lane's dims of head x (tile 0) / head x + 8 (tile 1)
  uint32_t qb0[NH][8], qb2[NH][8];
  float inv_s[NH], ksum[2 * NH];   // c2 / scale of head x (+8); 8 * sum_c q'[c] of heads 2t, 2t+1 (+8)
  float inv2[2 * NH];              // c2 / scale of heads 2t, 2t+1 (+8)
  int cur_prob = -1;
  const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(p.q);
  const float c2 = p.sm_scale * kLog2e;

  auto load_q_row = [&](int b, int hq, bool valid, uint32_t (&a0)[8], uint32_t (&a2)[8], float &inv, float &sum8) {
    uint4 v[4] = {};
    if (valid) {
      const uint4 *qp = reinterpret_cast<const uint4 *>(q + ((int64_t)b * p.Hq + hq) * LOCKS_D + 32 * t);
#pragma unroll
      for (int m = 0; m < 4; ++m) v[m] = __ldg(qp + m);
    }
    const uint32_t *w = reinterpret_cast<const uint32_t *>(v);
    uint32_t mx = 0u;  // largest |q| of the row as a bf16 bit pattern (orders like the value)
#pragma unroll
    for (int i = 0; i < 16; ++i) mx = __vmaxu2(mx, w[i] & 0x7FFF7FFFu);
    mx = max(mx & 0xFFFFu, mx >> 16);
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float fm = __uint_as_float(mx << 16);
    float s = 1.f;
    if (fm > 0.f && fm < INFINITY) {
      int e;
      (void)frexpf(fm, &e);        // fm = f 2^e, f in [0.5, 1)
      s = ldexpf(1.f, -(e + 1));   // max |q| s < 0.5
    }
    inv = 1.f / s;
    const float s16 = s * 0.0625f;
    float acc = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t u0 = w[2 * ks], u1 = w[2 * ks + 1];
      const uint32_t h0 = pack_f16(__uint_as_float(u0 << 16) * s, __uint_as_float(u0 & 0xFFFF0000u) * s);
      const uint32_t h1 = pack_f16(__uint_as_float(u1 << 16) * s, __uint_as_float(u1 & 0xFFFF0000u) * s);
      const float2 f0 = h2f2(h0), f1 = h2f2(h1);
      acc += (f0.x + f0.y) + (f1.x + f1.y);     // sum of the fp16 values actually multiplied
      a0[ks] = h0;
      a2[ks] = pack_f16(f1.x * 0.0625f, f1.y * 0.0625f);
    }
    (void)s16;
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    sum8 = 8.f * acc;
  };

  // candidate partial (max, sum exp) of the current problem, kept per lane and reduced across the warp
  // only when the warp moves on: one (head, warp) partial per problem instead of one per group
  float pm[NH], ps[NH];
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) { pm[hh] = -INFINITY; ps[hh] = 0.f; }
  int cur_b = 0, cur_h = 0, cur_pslot = sub;   // partial slot of this warp in the current problem
  float *srow[NH];                              // score row(s) of this lane's head(s) of the current problem
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) srow[hh] = p.shat;
  auto accumulate = [&](float &m, float &sacc, float v) {   // online log-sum-exp, one exp per value
    // branch-free: a value of -inf (masked page) adds nothing, whatever m is (also -inf at the start)
    const bool live = v > -INFINITY;
    const float d = v - m;                                    // NaN only if both are -inf: not live then
    const float e = live ? __expf(-fabsf(d)) : 0.f;           // m = -inf, v finite: exp(-inf) = 0
    const bool up = live && d > 0.f;
    sacc = up ? fmaf(sacc, e, 1.f) : sacc + e;
    m = up ? v : m;
  };
  float2 *red = reinterpret_cast<float2 *>(smem + kScanWarps * (kScanStages * kStageBytes + 64));   // [warp][16]
  auto flush = [&](bool to_smem, bool finished) {
    const int pslot = cur_pslot;
    // balanced: the warp that finishes a problem's last group knows how many partials it has
    if (BAL && finished && lane == 0) p.part_cnt[cur_prob] = pslot + 1;
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      float m = pm[hh], sacc = ps[hh];
#pragma unroll
      for (int o = 1; o <= 16; o <<= 1) {
        if (o == 4 || o == 8 || (o == 16 && !PK)) continue;   // lanes sharing a head: t (1, 2) and, packed, x bit 2
        const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, sacc, o);
        const float nm = fmaxf(m, om);
        if (nm > -INFINITY) { sacc = sacc * __expf(m - nm) + os * __expf(om - nm); m = nm; }
      }
      const int g = PK ? (x & 3) : x + 8 * hh;
      if (t == 0 && (!PK || x < 4) && g < p.G) {
        if (CR && to_smem) red[warp * 16 + g] = make_float2(m, sacc);
        else p.part[((int64_t)cur_b * p.Hq + cur_h * p.G + g) * p.max_groups + pslot] = make_float2(m, sacc);
      }
      pm[hh] = -INFINITY;
      ps[hh] = 0.f;
    }
  };

  int it = 0;
  bool ok = true;
  while (cc.prob < nprob) {
    const int stage = it % kScanStages;
    const uint32_t parity = (it / kScanStages) & 1;
    const int b = cc.b, h = cc.h;
    // a new problem's query is fetched and normalised BEFORE waiting for the group's summaries, so that the
    // round trip of the query load runs beside the copy instead of after it
    if (cc.prob != cur_prob) {
      if (cur_prob >= 0) flush(false, true);
      cur_prob = cc.prob;
      cur_b = b;
      cur_h = h;
      cur_pslot = BAL ? (it == 0 ? pslot_first : 0) : sub;
#pragma unroll
      for (int hh = 0; hh < NH; ++hh)
        srow[hh] = p.shat + ((int64_t)b * p.Hq + h * p.G + (PK ? (x & 3) : x + 8 * hh)) * p.Pmax;
#pragma unroll
      for (int hh = 0; hh < NH; ++hh) {
        float s8;
        const int gx = PK ? (x & 3) : x + 8 * hh;   // head held by this lane's column
        load_q_row(b, h * p.G + gx, gx < p.G, qb0[hh], qb2[hh], inv_s[hh], s8);
        // lane (x, t) owns head gx; the column fragment needs the heads of columns 2t, 2t+1
        ksum[2 * hh] = __shfl_sync(0xffffffffu, s8, (2 * t) * 4);
        ksum[2 * hh + 1] = __shfl_sync(0xffffffffu, s8, (2 * t + 1) * 4);
        inv_s[hh] *= c2;   // from here on: the factor that turns a scaled dot product into a log2-domain logit
        inv2[2 * hh] = __shfl_sync(0xffffffffu, inv_s[hh], (2 * t) * 4);
        inv2[2 * hh + 1] = __shfl_sync(0xffffffffu, inv_s[hh], (2 * t + 1) * 4);
      }
    }
    if (kScanBulk) {
      if (!mbar_wait(&full[stage], parity)) {
        ok = false;
        break;
      }
    } else {
      // groups complete in order: all but the newest (kScanStages - 1) committed groups must have landed
      if (inflight >= kScanStages) cp_async_wait<kScanStages - 1>(); else cp_async_wait<0>();
      __syncwarp();
    }
    --inflight;

    const uint8_t *sb = ring + stage * kStageBytes;
    // ---- centroid dots of the 8 pages.  Pages are the MMA rows (rows 8-15 idle) and the query is the B operand,
    // the same register pairs MMA #1 uses: cenT[hh][0..1] = sum_c code_mu[page x][c] q'[head 2t, 2t+1 (+8 hh)][c]
    float cenT[NH][4];
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) cenT[hh][0] = cenT[hh][1] = cenT[hh][2] = cenT[hh][3] = 0.f;
    {
      const uint4 *mp = reinterpret_cast<const uint4 *>(sb + boff(x & (LOCKS_GROUP - 1)) + i4_off_mu(R) + t * 32);
      const uint4 m0 = mp[0], m1 = mp[1];
      const uint32_t mw[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const uint32_t w = mw[s];
        const uint32_t b0 = f16x2_sub(and_or(w, kMB, kMagic), kSub128);              // code
        const uint32_t b1 = f16x2_fma(and_or(w >> 8, kMB, kMagic), kSixteen, kNeg16x);  // 16 * code
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) mma_f16(cenT[hh], b0, 0u, b1, 0u, qb0[hh][s], qb2[hh][s]);
      }
    }
    // scaled at the lane that holds them (page x, heads 2t, 2t+1), then moved to the lanes that finish the pages
    float acen[2 * NH];  // log2-domain centroid term: packed, of this lane's (page, head); else of pages 2t, 2t+1 for head x (+8)
    {
      const float smu = __half2float(*reinterpret_cast<const __half *>(sb + boff(x & (LOCKS_GROUP - 1)) + i4_off_smu(R)));
#pragma unroll
      for (int hh = 0; hh < NH; ++hh) {
        const float v0 = smu * inv2[2 * hh] * cenT[hh][0], v1 = smu * inv2[2 * hh + 1] * cenT[hh][1];
        if (PK) {   // lane (x, t) finishes page 2t + (x >> 2), head x & 3: held by lane (that page, (x & 3) >> 1)
          const int src = (2 * t + (x >> 2)) * 4 + ((x & 3) >> 1);
          const float a0 = __shfl_sync(0xffffffffu, v0, src), a1 = __shfl_sync(0xffffffffu, v1, src);
          acen[0] = (x & 1) ? a1 : a0;
          acen[1] = 0.f;
        } else {    // lane (x, t) finishes pages 2t, 2t + 1 for head x (+8 hh): held by lanes (page, x >> 1)
          const int srcA = (2 * t) * 4 + (x >> 1), srcB = srcA + 4;
          const float a0 = __shfl_sync(0xffffffffu, v0, srcA), a1 = __shfl_sync(0xffffffffu, v1, srcA);
          const float b0 = __shfl_sync(0xffffffffu, v0, srcB), b1 = __shfl_sync(0xffffffffu, v1, srcB);
          acen[2 * hh] = (x & 1) ? a1 : a0;
          acen[2 * hh + 1] = (x & 1) ? b1 : b0;
        }
      }
    }
    float res[2 * NH];
#pragma unroll
    for (int i = 0; i < 2 * NH; ++i) res[i] = 0.f;

    float prj2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};   // small-rank tile: projections of the current MMA #1 chain
    (void)prj2;
    if constexpr (R <= 4 && PK) {
      // ---- ranks 2 and 4, G <= 4.  MMA #1: the 16 rows are (page, rank) pairs, 8 / R pages in rows 0-7 and the
      // next 8 / R in rows 8-15, so one chain of 8 MMAs projects 16 / R pages (rank 2: the whole group; rank 4:
      // half of it); lane (x, t) loads the quarter-t words of its (page, rank).  MMA #2 works on four pages at a
      // time: rows = (page a, head g) = 4 a + g, columns = tokens, k = (page, rank) so that a row meets its own
      // page only (block diagonal).  Rank 2: k = part * 8 + 2 a + rank with part 0 / 1 = fp16 hi / lo of the
      // projection, one MMA per token half.  Rank 4: k = 4 a + rank, hi and lo in two MMAs.
      constexpr int PH = 8 / R;                 // pages per row half of MMA #1
      const int pr = x / R, lr = x % R;         // this lane's row: page within the half, rank
      const float iv = inv_s[0];
#pragma unroll
      for (int k4 = 0; k4 < 2; ++k4) {          // pages 4 k4 .. 4 k4 + 3
        float prj[2][2];                        // rank 2: [k4 half][head e]; rank 4: [half of this chain][head e]
        if (R == 4 || k4 == 0) {
          const int pa0 = (R == 4 ? 4 * k4 : 0) + pr, pb0 = pa0 + PH;
          const uint4 wa4 = *reinterpret_cast<const uint4 *>(sb + boff(pa0) + (lr * 4 + t) * 16);
          const uint4 wb4 = *reinterpret_cast<const uint4 *>(sb + boff(pb0) + (lr * 4 + t) * 16);
          const uint32_t wa[4] = {wa4.x, wa4.y, wa4.z, wa4.w}, wb[4] = {wb4.x, wb4.y, wb4.z, wb4.w};
          float c1[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t ua = wa[j], ub = wb[j], ua8 = ua >> 8, ub8 = ub >> 8;
            if (j == 0) mma_f16_z(c1, ua & kM0, ub & kM0, ua & kM1, ub & kM1, qb0[0][0], qb2[0][0]);
            else mma_f16(c1, ua & kM0, ub & kM0, ua & kM1, ub & kM1, qb0[0][2 * j], qb2[0][2 * j]);
            mma_f16(c1, ua8 & kM0, ub8 & kM0, ua8 & kM1, ub8 & kM1, qb0[0][2 * j + 1], qb2[0][2 * j + 1]);
          }
          const float svA = __half2float(*reinterpret_cast<const __half *>(sb + boff(pa0) + i4_off_sv(R) + 2 * lr));
          const float svB = __half2float(*reinterpret_cast<const __half *>(sb + boff(pb0) + i4_off_sv(R) + 2 * lr));
          prj2[0][0] = fmaf(c1[0], 16777216.f, -ksum[0]) * svA;
          prj2[0][1] = fmaf(c1[1], 16777216.f, -ksum[1]) * svA;
          prj2[1][0] = fmaf(c1[2], 16777216.f, -ksum[0]) * svB;
          prj2[1][1] = fmaf(c1[3], 16777216.f, -ksum[1]) * svB;
        }
        prj[0][0] = prj2[0][0]; prj[0][1] = prj2[0][1]; prj[1][0] = prj2[1][0]; prj[1][1] = prj2[1][1];
        uint32_t a0h, a1h, a2h, a3h, a0l = 0u, a1l = 0u, a2l = 0u, a3l = 0u;
        uint32_t bt0a, bt0b, bt8a, bt8b;
        if (R == 2) {
          // lane (x, t) feeds page t of the four, head x & 3, if its row x (t < 2) or x + 8 (t >= 2) is that page's
          const bool mine = (x >> 2) == (t & 1);
          const int src0 = (2 * t) * 4 + ((x & 3) >> 1), src1 = src0 + 4;   // lanes holding rank 0 | 1 of (page t, head pair)
          const float r00 = __shfl_sync(0xffffffffu, prj[k4][0], src0), r01 = __shfl_sync(0xffffffffu, prj[k4][1], src0);
          const float r10 = __shfl_sync(0xffffffffu, prj[k4][0], src1), r11 = __shfl_sync(0xffffffffu, prj[k4][1], src1);
          const float p0 = (x & 1) ? r01 : r00, p1 = (x & 1) ? r11 : r10;   // ranks 0, 1 of (page t, head x & 3)
          uint32_t hi = pack_f16(p0, p1);
          const float2 hf = h2f2(hi);
          uint32_t lo = pack_f16(p0 - hf.x, p1 - hf.y);
          if (!mine) { hi = 0u; lo = 0u; }
          a0h = t < 2 ? hi : 0u; a1h = t < 2 ? 0u : hi; a2h = t < 2 ? lo : 0u; a3h = t < 2 ? 0u : lo;
          // coefficients of page t, token x (and x + 8), ranks 0 and 1; the lo part meets the same values
          const uint32_t cw = *reinterpret_cast<const uint32_t *>(sb + boff(4 * k4 + t) + i4_off_coef(R) + x * 4);
          bt0a = bt0b = f16x2_sub(__byte_perm(cw, 0x64646464u, 0x4140), kSub128);
          bt8a = bt8b = f16x2_sub(__byte_perm(cw, 0x64646464u, 0x4342), kSub128);
        } else {
          // k = 2t, 2t+1 is (page t >> 1, ranks 2 (t & 1), + 1) of pages 0-1, k + 8 the same of pages 2-3; rows x are
          // pages 0-1 (page x >> 2), rows x + 8 pages 2-3: a0 and a3 carry the diagonal blocks, a1 = a2 = 0
          const bool mine = (x >> 2) == (t >> 1);
          const int src0 = ((x >> 2) * 4 + 2 * (t & 1)) * 4 + ((x & 3) >> 1), src1 = src0 + 4;
          float pv[2][2];   // [half][rank of the pair]
#pragma unroll
          for (int hf2 = 0; hf2 < 2; ++hf2) {
            const float r00 = __shfl_sync(0xffffffffu, prj[hf2][0], src0), r01 = __shfl_sync(0xffffffffu, prj[hf2][1], src0);
            const float r10 = __shfl_sync(0xffffffffu, prj[hf2][0], src1), r11 = __shfl_sync(0xffffffffu, prj[hf2][1], src1);
            pv[hf2][0] = (x & 1) ? r01 : r00;
            pv[hf2][1] = (x & 1) ? r11 : r10;
          }
          uint32_t hi0 = pack_f16(pv[0][0], pv[0][1]), hi1 = pack_f16(pv[1][0], pv[1][1]);
          const float2 f0 = h2f2(hi0), f1 = h2f2(hi1);
          uint32_t lo0 = pack_f16(pv[0][0] - f0.x, pv[0][1] - f0.y), lo1 = pack_f16(pv[1][0] - f1.x, pv[1][1] - f1.y);
          if (!mine) { hi0 = hi1 = lo0 = lo1 = 0u; }
          a0h = hi0; a1h = 0u; a2h = 0u; a3h = hi1;
          a0l = lo0; a3l = lo1;
          const int wofs = i4_off_coef(R) + (x * 2 + (t & 1)) * 4;   // token x (and x + 8), rank pair t & 1
          const uint32_t cw0 = *reinterpret_cast<const uint32_t *>(sb + boff(4 * k4 + (t >> 1)) + wofs);
          const uint32_t cw1 = *reinterpret_cast<const uint32_t *>(sb + boff(4 * k4 + 2 + (t >> 1)) + wofs);
          bt0a = f16x2_sub(__byte_perm(cw0, 0x64646464u, 0x4140), kSub128);
          bt0b = f16x2_sub(__byte_perm(cw1, 0x64646464u, 0x4140), kSub128);
          bt8a = f16x2_sub(__byte_perm(cw0, 0x64646464u, 0x4342), kSub128);
          bt8b = f16x2_sub(__byte_perm(cw1, 0x64646464u, 0x4342), kSub128);
        }
        float ca[4], cb[4];   // ca: tokens 2t, 2t+1; cb: tokens 2t+8, 2t+9; [0..1] row x, [2..3] row x + 8
        mma_f16_z(ca, a0h, a1h, a2h, a3h, bt0a, bt0b);
        mma_f16_z(cb, a0h, a1h, a2h, a3h, bt8a, bt8b);
        if (R == 4) {
          mma_f16(ca, a0l, a1l, a2l, a3l, bt0a, bt0b);
          mma_f16(cb, a0l, a1l, a2l, a3l, bt8a, bt8b);
        }
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {   // row x -> page 4 k4 + (x >> 2), row x + 8 -> two pages further
          const int pg = 4 * k4 + 2 * hrow + (x >> 2);
          const uint2 scw = *reinterpret_cast<const uint2 *>(sb + boff(pg) + i4_off_sc(R) + 8 * t);
          const float2 s01 = h2f2(scw.x), s89 = h2f2(scw.y);
          const float y0 = ca[2 * hrow] * s01.x, y1 = ca[2 * hrow + 1] * s01.y;
          const float y2 = cb[2 * hrow] * s89.x, y3 = cb[2 * hrow + 1] * s89.y;
          float my = fmaxf(fmaxf(y0, y1), fmaxf(y2, y3));
          my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 1));
          my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 2));
          const float m = my * iv;
          float e = fast_ex2(fmaf(y0, iv, -m)) + fast_ex2(fmaf(y1, iv, -m)) + fast_ex2(fmaf(y2, iv, -m)) +
                    fast_ex2(fmaf(y3, iv, -m));
          e += __shfl_xor_sync(0xffffffffu, e, 1);
          e += __shfl_xor_sync(0xffffffffu, e, 2);
          // lane (x, t) keeps the result of page 2t + (x >> 2), head x & 3
          if (t == 2 * k4 + hrow) res[0] = m + fast_lg2(e) + acen[0];
        }
      }
    } else {
#pragma unroll
    for (int pp = 0; pp < LOCKS_GROUP / 2; ++pp) {
      const uint8_t *pbA = sb + boff(2 * pp), *pbB = pbA + kBlob;
      // ---- MMA #1: rows = (page A ranks 0-7, page B ranks 0-7), cols = heads, k = this lane quarter's dims
      // lane (x, t) holds rank x, dim quarter t; ranks >= R do not exist (their column scale reads as 0 below)
      const uint4 wa4 = (R == 8 || x < R) ? *reinterpret_cast<const uint4 *>(pbA + lane * 16) : make_uint4(0u, 0u, 0u, 0u);
      const uint4 wb4 = (R == 8 || x < R) ? *reinterpret_cast<const uint4 *>(pbB + lane * 16) : make_uint4(0u, 0u, 0u, 0u);
      const uint32_t wa[4] = {wa4.x, wa4.y, wa4.z, wa4.w}, wb[4] = {wb4.x, wb4.y, wb4.z, wb4.w};
      float c1[NH][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t ua = wa[j], ub = wb[j], ua8 = ua >> 8, ub8 = ub >> 8;
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
          if (j == 0) mma_f16_z(c1[hh], ua & kM0, ub & kM0, ua & kM1, ub & kM1, qb0[hh][0], qb2[hh][0]);
          else mma_f16(c1[hh], ua & kM0, ub & kM0, ua & kM1, ub & kM1, qb0[hh][2 * j], qb2[hh][2 * j]);
          mma_f16(c1[hh], ua8 & kM0, ub8 & kM0, ua8 & kM1, ub8 & kM1, qb0[hh][2 * j + 1], qb2[hh][2 * j + 1]);
        }
      }
      if (PK) {
        // lanes t < 2 carry page A (columns 0-3), lanes t >= 2 page B (columns 4-7)
        const bool pa = t < 2;
        const uint8_t *pbs = pa ? pbA : pbB;
        const float sv = (R == 8 || x < R) ? __half2float(*reinterpret_cast<const __half *>(pbs + i4_off_sv(R) + 2 * x)) : 0.f;
        const float p0 = fmaf(pa ? c1[0][0] : c1[0][2], 16777216.f, -ksum[0]) * sv;
        const float p1 = fmaf(pa ? c1[0][1] : c1[0][3], 16777216.f, -ksum[1]) * sv;
        const uint32_t hi = pack_f16(p0, p1);
        const float2 hf = h2f2(hi);
        const uint32_t lo = pack_f16(p0 - hf.x, p1 - hf.y);
        const uint32_t hiT = movm_trans(hi), loT = movm_trans(lo);   // lane (x, t): row x, ranks 2t, 2t+1
        const bool ra = x < 4;                                        // row x: page A head x | page B head x - 4
        const uint32_t hA = ra ? hiT : 0u, hB = ra ? 0u : hiT, lA = ra ? loT : 0u, lB = ra ? 0u : loT;
        // lane (x, t): tokens x and x + 8, ranks 2t and 2t + 1; missing rank pairs read as code 0
        const uint32_t cwa = (t < R / 2) ? *reinterpret_cast<const uint32_t *>(pbA + i4_off_coef(R) + (x * (R / 2) + t) * 4) : 0x80808080u;
        const uint32_t cwb = (t < R / 2) ? *reinterpret_cast<const uint32_t *>(pbB + i4_off_coef(R) + (x * (R / 2) + t) * 4) : 0x80808080u;
        const uint32_t a0 = f16x2_sub(__byte_perm(cwa, 0x64646464u, 0x4140), kSub128);
        const uint32_t a1 = f16x2_sub(__byte_perm(cwa, 0x64646464u, 0x4342), kSub128);
        const uint32_t b0 = f16x2_sub(__byte_perm(cwb, 0x64646464u, 0x4140), kSub128);
        const uint32_t b1 = f16x2_sub(__byte_perm(cwb, 0x64646464u, 0x4342), kSub128);
        // k 0-7 = page A's ranks, k 8-15 = page B's ranks; hi and lo parts accumulate into the same tile
        float ca[4], cb[4];
        mma_f16_z(ca, hA, 0u, hB, 0u, a0, b0);
        mma_f16(ca, lA, 0u, lB, 0u, a0, b0);
        mma_f16_z(cb, hA, 0u, hB, 0u, a1, b1);
        mma_f16(cb, lA, 0u, lB, 0u, a1, b1);
        const uint2 scw = *reinterpret_cast<const uint2 *>((ra ? pbA : pbB) + i4_off_sc(R) + 8 * t);
        const float2 s01 = h2f2(scw.x), s89 = h2f2(scw.y);
        const float iv = inv_s[0];
        const float y0 = ca[0] * s01.x, y1 = ca[1] * s01.y, y2 = cb[0] * s89.x, y3 = cb[1] * s89.y;
        float my = fmaxf(fmaxf(y0, y1), fmaxf(y2, y3));
        my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 1));
        my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 2));
        const float m = my * iv;
        float e = fast_ex2(fmaf(y0, iv, -m)) + fast_ex2(fmaf(y1, iv, -m)) + fast_ex2(fmaf(y2, iv, -m)) +
                  fast_ex2(fmaf(y3, iv, -m));
        e += __shfl_xor_sync(0xffffffffu, e, 1);
        e += __shfl_xor_sync(0xffffffffu, e, 2);
        // lane (x, t = pp) keeps the result of page 2 pp + (x >> 2), head x & 3
        if (t == pp) res[0] = m + fast_lg2(e) + acen[0];
      } else {
#pragma unroll
      for (int pq = 0; pq < 2; ++pq) {
        const int pg = 2 * pp + pq;
        const uint8_t *pb = pq ? pbB : pbA;
        // projection of rank x for heads 2t, 2t+1: undo 2^-24, remove the +8 offset, apply the column scale
        const float sv = (R == 8 || x < R) ? __half2float(*reinterpret_cast<const __half *>(pb + i4_off_sv(R) + 2 * x)) : 0.f;
        uint32_t hiT[NH], loT[NH];
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
          const float p0 = fmaf(c1[hh][2 * pq], 16777216.f, -ksum[2 * hh]) * sv;
          const float p1 = fmaf(c1[hh][2 * pq + 1], 16777216.f, -ksum[2 * hh + 1]) * sv;
          const uint32_t hi = pack_f16(p0, p1);
          const float2 hf = h2f2(hi);
          const uint32_t lo = pack_f16(p0 - hf.x, p1 - hf.y);
          hiT[hh] = movm_trans(hi);   // -> lane (x = head, t): ranks 2t, 2t+1
          loT[hh] = movm_trans(lo);
        }
        // ---- MMA #2: rows = heads, k = ranks (hi | lo), cols = tokens
        const uint32_t cw = (t < R / 2) ? *reinterpret_cast<const uint32_t *>(pb + i4_off_coef(R) + (x * (R / 2) + t) * 4) : 0x80808080u;
        const uint32_t b0 = f16x2_sub(__byte_perm(cw, 0x64646464u, 0x4140), kSub128);
        const uint32_t b1 = f16x2_sub(__byte_perm(cw, 0x64646464u, 0x4342), kSub128);
        float ca[4], cb[4];
        mma_f16_z(ca, hiT[0], NH == 2 ? hiT[NH - 1] : 0u, loT[0], NH == 2 ? loT[NH - 1] : 0u, b0, b0);
        mma_f16_z(cb, hiT[0], NH == 2 ? hiT[NH - 1] : 0u, loT[0], NH == 2 ? loT[NH - 1] : 0u, b1, b1);
        const uint2 scw = *reinterpret_cast<const uint2 *>(pb + i4_off_sc(R) + 8 * t);
        const float2 s01 = h2f2(scw.x), s89 = h2f2(scw.y);
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
          const float iv = inv_s[hh];   // logits (log2 domain) are y * iv, iv > 0
          const float y0 = ca[2 * hh] * s01.x, y1 = ca[2 * hh + 1] * s01.y;
          const float y2 = cb[2 * hh] * s89.x, y3 = cb[2 * hh + 1] * s89.y;
          float my = fmaxf(fmaxf(y0, y1), fmaxf(y2, y3));
          my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 1));
          my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 2));
          const float m = my * iv;
          float e = fast_ex2(fmaf(y0, iv, -m)) + fast_ex2(fmaf(y1, iv, -m)) + fast_ex2(fmaf(y2, iv, -m)) +
                    fast_ex2(fmaf(y3, iv, -m));
          e += __shfl_xor_sync(0xffffffffu, e, 1);
          e += __shfl_xor_sync(0xffffffffu, e, 2);
          const float v = m + fast_lg2(e);
          if (t == (pg >> 1)) res[2 * hh + (pg & 1)] = v;
        }
      }
    }
      }
    }
    __syncwarp();  // every lane is done reading this stage
    if (cp.prob < nprob) {
      issue(stage, cp, next_block);
      ++inflight;
      advance(cp, it + 1 + inflight < n_units);
      next_block = fetch_block(cp);
    }

    // ---- write s^ and the group's candidate partial
    if (PK) {
      const int g = x & 3, page = cc.grp * LOCKS_GROUP + 2 * t + (x >> 2);
      const float v = res[0] * kLn2;
      const bool in = t < LOCKS_GROUP / 2 && page < cc.nsc;
      if (g < p.G && in) store_score(srow[0] + page, v);
      accumulate(pm[0], ps[0], (in && page >= 1) ? v : -INFINITY);
    } else {
    const int page0 = cc.grp * LOCKS_GROUP + 2 * t;
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      const int g = x + 8 * hh;
      const float v0 = (res[2 * hh] + acen[2 * hh]) * kLn2;
      const float v1 = (res[2 * hh + 1] + acen[2 * hh + 1]) * kLn2;
      const bool in0 = t < LOCKS_GROUP / 2 && page0 < cc.nsc, in1 = t < LOCKS_GROUP / 2 && page0 + 1 < cc.nsc;
      if (g < p.G) {
        float *dst = srow[hh] + page0;
        if (in0) store_score(dst, v0);
        if (in1) store_score(dst + 1, v1);
      }
      accumulate(pm[hh], ps[hh], (in0 && page0 >= 1) ? v0 : -INFINITY);
      accumulate(pm[hh], ps[hh], in1 ? v1 : -INFINITY);
    }
    }
    advance(cc, it + 1 < n_units);
    ++it;
  }
  if (CR) {
    // geometry guarantees that all warps of this CTA reach this point and share the problem `slot`
    flush(true, true);
    __syncthreads();
    if (warp == 0 && lane < p.G) {
      float m = -INFINITY, sacc = 0.f;
#pragma unroll
      for (int w = 0; w < kScanWarps; ++w) {
        const float2 v = red[w * 16 + lane];
        const float nm = fmaxf(m, v.x);
        if (nm > -INFINITY) { sacc = sacc * __expf(m - nm) + v.y * __expf(v.x - nm); m = nm; }
      }
      const int pb = slot / p.Hkv, ph = slot - pb * p.Hkv;
      p.part[((int64_t)pb * p.Hq + ph * p.G + lane) * p.max_groups + sub / kScanWarps] = make_float2(m, sacc);
    }
  } else if (ok && cur_prob >= 0) {
    flush(false, cc.grp * LOCKS_GROUP >= cc.nsc);   // the last unit was the problem's last group
  }
  if (!ok) {
    // a wait ran out: flag it, then give copies still in flight a bounded chance to land before exit
    if (lane == 0) set_status(p.status, LOCKS_ERR_TIMEOUT);
    for (int s = 0; s < inflight && s < kScanStages; ++s) {
      const int st = (it + s) % kScanStages;
      (void)mbar_wait(&full[st], ((it + s) / kScanStages) & 1);
    }
  }
}

}  // namespace

locks_scan_geom locks_scan_geometry(const locks_ctx *c, int batch) {
  locks_scan_geom g;
  const int Hkv = c->cfg.num_kv_heads;
  const int total_groups = batch * Hkv * c->max_groups;
  g.grid = kScanCtasPerSm * c->num_sms;
  const int need = (total_groups + kScanWarps - 1) / kScanWarps;
  if (g.grid > need) g.grid = need < 1 ? 1 : need;
  g.W = g.grid * kScanWarps;
  const int nprob = batch * Hkv;
  g.wpp = g.W / nprob > 1 ? g.W / nprob : 1;
  g.nslots = g.W / g.wpp;
  g.rounds = (nprob + g.nslots - 1) / g.nslots;
  // few problems: every CTA's warps share one problem for the whole launch and none leaves early,
  // so the CTA merges its warps' partials before writing (the selector reads 8x fewer)
  g.cta_reduce = (c->cfg.rank == 8 && g.wpp % kScanWarps == 0 && g.nslots == nprob && g.nslots * g.wpp == g.W) ? 1 : 0;
  return g;
}

int locks_launch_scan(locks_ctx *c, const void *q, const void *summaries, const locks_kv *kv, int batch,
                      float *shat, int seq_inc, cudaStream_t st) {
  ScanParams p;
  p.cta_reduce = 0;
  p.seq_inc = seq_inc;
  p.seq_eff = seq_inc ? c->seq_eff : nullptr;
  p.q = q;
  p.summ = reinterpret_cast<const uint8_t *>(summaries);
  p.block_table = kv->block_table;
  p.seq_lens = kv->seq_lens;
  p.shat = shat;
  p.part = c->part;
  p.part_cnt = c->part_cnt;
  p.status = c->status;
  p.batch = batch; p.Hq = c->cfg.num_q_heads; p.Hkv = c->cfg.num_kv_heads; p.G = c->G;
  p.Pmax = c->Pmax; p.max_groups = c->max_groups; p.num_blocks = kv->num_blocks; p.k = c->k;
  p.S = c->S; p.r = c->cfg.rank; p.sm_scale = c->cfg.sm_scale; p.B = c->B;
  p.scorer = c->scorer;
  const bool tensor = c->cfg.summary_fmt == LOCKS_FMT_I4 && c->cfg.q_dtype == LOCKS_BF16 &&
                      c->scorer == LOCKS_SCORER_SUMMARY && c->B == LOCKS_B;   // ranks 2, 4, 8
  c->part_slots = c->max_groups;   // generic kernel: one partial per 8-page group
  c->part_balanced = 0;
  c->last_partition = 0;
  if (tensor) {
    const locks_scan_geom geo = locks_scan_geometry(c, batch);
    const int grid = geo.grid;
    p.wpp = geo.wpp; p.nslots = geo.nslots; p.cta_reduce = geo.cta_reduce;
    // strided partition: one partial per (problem, warp), or per (problem, CTA) with the CTA-level merge;
    // balanced partition: the kernel counts the partials of each problem itself (part_cnt)
    c->part_slots = geo.cta_reduce ? geo.wpp / kScanWarps : geo.wpp;
    int mode = c->scan_partition;
    if (mode == LOCKS_PARTITION_AUTO)
      mode = (c->hint_host && *reinterpret_cast<volatile int32_t *>(c->hint_host) == LOCKS_PARTITION_BALANCED)
                 ? LOCKS_PARTITION_BALANCED : LOCKS_PARTITION_STRIDED;
    // the balanced partition also replaces the CTA-level merge of the few-problem geometry when it is asked for:
    // a few requests of very different lengths would otherwise leave most of the GPU waiting for the longest
    const bool balanced = LOCKS_SCAN_BALANCED && mode == LOCKS_PARTITION_BALANCED;
    if (balanced) {
      p.cta_reduce = 0;
      c->part_slots = geo.wpp;
    }
    c->part_balanced = balanced ? 1 : 0;
    c->last_partition = balanced ? LOCKS_PARTITION_BALANCED : LOCKS_PARTITION_STRIDED;
    const dim3 g(grid), blk(kScanWarps * 32);
    const int gsel = c->G <= 4 ? 0 : (c->G <= 8 ? 1 : 2);
    // tensor map over the summaries for the gather path: rows = (block, KV head), S / 4 32-bit words each
    alignas(64) CUtensorMap tmap;
    memset(&tmap, 0, sizeof(tmap));
    p.use_gather = 0;
    if (LOCKS_SCAN_GATHER) {
      static PFN_cuTensorMapEncodeTiled encode = nullptr;
      static bool looked = false;
      if (!looked) {
        looked = true;
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
          encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
        (void)cudaGetLastError();
      }
      if (encode) {
        const int S = i4_stride(c->cfg.rank);
        const cuuint64_t gdim[2] = {(cuuint64_t)(S / 4), (cuuint64_t)kv->num_blocks * p.Hkv};
        const cuuint64_t gstride[1] = {(cuuint64_t)S};
        const cuuint32_t box[2] = {(cuuint32_t)(S / 4), 1u};
        const cuuint32_t estride[2] = {1u, 1u};
        if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(summaries), gdim, gstride, box, estride,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
          p.use_gather = 1;
      }
    }
#define LOCKS_SCAN_LAUNCH(R_, CR_, BAL_)                                                                                  \
  do {                                                                                                                 \
    if (locks_attrs_needed(LOCKS_ATTR_SCAN + (R_ == 8 ? 0 : (R_ == 4 ? 4 : 8)) + (CR_ ? 2 : 0) + (BAL_ ? 1 : 0))) {     \
      cudaFuncSetAttribute(scan_i4_kernel<R_, 1, true, CR_, BAL_>, cudaFuncAttributeMaxDynamicSharedMemorySize, kScanSmem);  \
      cudaFuncSetAttribute(scan_i4_kernel<R_, 1, false, CR_, BAL_>, cudaFuncAttributeMaxDynamicSharedMemorySize, kScanSmem); \
      cudaFuncSetAttribute(scan_i4_kernel<R_, 2, false, CR_, BAL_>, cudaFuncAttributeMaxDynamicSharedMemorySize, kScanSmem); \
    }                                                                                                                  \
    if (gsel == 0) locks_launch_pdl(scan_i4_kernel<R_, 1, true, CR_, BAL_>, g, blk, kScanSmem, st, p, tmap);                       \
    else if (gsel == 1) locks_launch_pdl(scan_i4_kernel<R_, 1, false, CR_, BAL_>, g, blk, kScanSmem, st, p, tmap);                 \
    else locks_launch_pdl(scan_i4_kernel<R_, 2, false, CR_, BAL_>, g, blk, kScanSmem, st, p, tmap);                                \
  } while (0)
    if (c->cfg.rank == 8 && p.cta_reduce) LOCKS_SCAN_LAUNCH(8, true, false);
    else if (c->cfg.rank == 8 && balanced) LOCKS_SCAN_LAUNCH(8, false, true);
    else if (c->cfg.rank == 8) LOCKS_SCAN_LAUNCH(8, false, false);
    else if (c->cfg.rank == 4 && balanced) LOCKS_SCAN_LAUNCH(4, false, true);
    else if (c->cfg.rank == 4) LOCKS_SCAN_LAUNCH(4, false, false);
    else if (balanced) LOCKS_SCAN_LAUNCH(2, false, true);
    else LOCKS_SCAN_LAUNCH(2, false, false);
#undef LOCKS_SCAN_LAUNCH
  } else {
    dim3 grid((c->max_groups + 3) / 4, p.Hkv, batch);
    const bool qbf = c->cfg.q_dtype == LOCKS_BF16;
    if (c->cfg.summary_fmt == LOCKS_FMT_F32) {
      if (qbf) locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_F32, __nv_bfloat16>, grid, dim3(128), 0, st, p);
      else locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_F32, float>, grid, dim3(128), 0, st, p);
    } else if (c->cfg.summary_fmt == LOCKS_FMT_I8) {
      if (qbf) locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_I8, __nv_bfloat16>, grid, dim3(128), 0, st, p);
      else locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_I8, float>, grid, dim3(128), 0, st, p);
    } else if (c->cfg.summary_fmt == LOCKS_FMT_BF16) {
      if (qbf) locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_BF16, __nv_bfloat16>, grid, dim3(128), 0, st, p);
      else locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_BF16, float>, grid, dim3(128), 0, st, p);
    } else {
      if (qbf) locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_I4, __nv_bfloat16>, grid, dim3(128), 0, st, p);
      else locks_launch_pdl(scan_generic_kernel<LOCKS_FMT_I4, float>, grid, dim3(128), 0, st, p);
    }
  }
  return locks_check_launch(c);
}
