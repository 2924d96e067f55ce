// Summary build (Sec. 4 "Build (once, when a page completes)").
//
// build_kernel: one warp takes 8 (page, KV head) items through three phases.
//   1. per item, all lanes: load the page's 16 keys (lane owns 4 consecutive dims of every key), centroid mu,
//      deviations D, and the Gram matrix M = D D^T (16 x 16) on the tensor cores; M goes to shared memory
//   2. all 8 items at once: eigendecomposition of M by one-sided Jacobi in fp32.  Four lanes hold one item's
//      matrix (4 columns of 16 entries each, in registers); columns are rotated in pairs until they are mutually
//      orthogonal, which leaves M W = U Lambda: column norms are the eigenvalues, normalised columns the
//      eigenvectors.  Pairing by odd-even transposition (16 steps per sweep meet every two columns once; a
//      rotated pair swaps places), so only the pairs that straddle two lanes need shuffles.
//   3. per item, all lanes: reload the keys, rank the modes by eigenvalue, keep r_eff <= min(r, 15) modes above
//      the zero-mode thresholds, V = D^T U_r Sigma_r^-1 (lane's 4 dims), C = U_r Sigma_r, sign: largest |V| entry
//      positive; store fp32 (F32 format) or quantise: symmetric abs-max, fp16 scale, round-half-even codes
//      (int4 basis per column, int8 coefficients per row, int8 centroid) packed in the blob layout
#include "locks_internal.cuh"

namespace {

struct BuildParams {
  const void *k;
  int64_t sb, sh, st;
  const int32_t *block_table;
  const int32_t *seq_lens;
  const int32_t *page_begin, *page_end;
  uint8_t *summ;
  int32_t *status;
  int batch, Hkv, Pmax, num_blocks, r, S, just_filled;
  // decode step only: where to leave the scan-partition suggestion for these lengths, and the scan's geometry
  int32_t *hint;
  int kpages, hint_wpp, hint_rounds, hint_W;
  // decode step only: the token appended by this step is read from the caller's buffer, not from the cache
  // (the append runs in another kernel at the same time); append_pos[b] = its position or -1
  const void *k_new;
  const int32_t *append_pos;
  // bulk build of several layers in one launch: per-layer key caches and summary buffers (device arrays), or null
  const void *const *k_layers;
  void *const *summ_layers;
};

#ifndef LOCKS_BUILD_COS_TOL
#define LOCKS_BUILD_COS_TOL 1e-3f   // a sweep that met no pair above this |cosine| was the last (it left them near 1e-6: quadratic convergence)
#endif
#ifndef LOCKS_BUILD_SWEEPS
#define LOCKS_BUILD_SWEEPS 16   // upper bound; the sweeps stop after one in which every pair of an item was orthogonal
#endif
constexpr int kBuildWarps = 2;
constexpr int kBuildItems = 8;                                   // (page, KV head) items per warp
#ifndef LOCKS_BUILD_CTAS
#define LOCKS_BUILD_CTAS 8
#endif
constexpr int kBuildCtasPerSm = LOCKS_BUILD_CTAS;                // 16 warps per SM
constexpr int kBuildScratch = 2 * LOCKS_B * 128;                 // 4096 B: bf16 half-tiles of D (hi | lo); later the blob
constexpr int kBuildMat = kBuildItems * LOCKS_B * LOCKS_B * 4;   // 8192 B: Gram matrices; later the leading eigenvectors, every entry twice
constexpr int kBuildSmemPerWarp = kBuildScratch + kBuildMat + 64 + kBuildItems * LOCKS_B * 4;   // + key norms, eigenvalues

// code = clamp(rint(x / scale)); `inv` = 1 / scale correctly rounded (0 for a zero scale: all codes 0).  The
// product differs from the quotient by at most an ulp, which matters only within an ulp of a rounding boundary.
__device__ __forceinline__ float inv_scale(float scale) { return scale == 0.f ? 0.f : __frcp_rn(scale); }
__device__ __forceinline__ float round_code(float x, float inv, float qmax) {
  return fminf(fmaxf(rintf(x * inv), -qmax), qmax);
}

// packed fp32 pairs (two independent lanes of arithmetic per instruction)
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(*reinterpret_cast<unsigned long long *>(&d))
      : "l"(*reinterpret_cast<unsigned long long *>(&a)), "l"(*reinterpret_cast<unsigned long long *>(&b)),
        "l"(*reinterpret_cast<unsigned long long *>(&c)));
  return d;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
  float2 d;
  asm("mul.rn.f32x2 %0, %1, %2;"
      : "=l"(*reinterpret_cast<unsigned long long *>(&d))
      : "l"(*reinterpret_cast<unsigned long long *>(&a)), "l"(*reinterpret_cast<unsigned long long *>(&b)));
  return d;
}

// The plane rotation that makes two columns p, q orthogonal, from a = |p|^2, b = |q|^2, g = p . q (smaller angle):
// with d = b - a and h = d^2 + 4 g^2, cos 2t = |d| / sqrt(h) and sin 2t = 2 g sign(d) / sqrt(h), so
// c = sqrt((1 + cos 2t) / 2) and s = sin 2t / (2 c): two reciprocal square roots in a row (approximate ones are
// enough for the angle; c^2 + s^2 = 1 holds to their rounding).  p' = c p - s q, q' = s p + c q.  Inputs too small
// or too large to square are left alone.
__device__ __forceinline__ float rsqrt_approx(float x) {
  float y;
  asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void jacobi_angle(float a, float b, float g, float &c, float &sn) {
  const float d = b - a, hh = fmaf(d, d, 4.f * g * g);
  const bool ok = hh > 1e-37f && hh < 1e37f;   // branch-free: independent pairs interleave in one basic block
  const float rs = rsqrt_approx(ok ? hh : 1.f);
  const float x = fmaf(0.5f * fabsf(d), rs, 0.5f);
  const float r2 = rsqrt_approx(x);
  const float s0 = copysignf(g * rs * r2, d == 0.f ? g : g * d);
  c = ok ? x * r2 : 1.f;
  sn = ok ? s0 : 0.f;
}

// One-sided Jacobi on 32 / LPI matrices at once, LPI = 16 / CPL lanes per matrix.  Lane (item = lane / LPI,
// j = lane % LPI) holds columns CPL j .. CPL j + CPL - 1 of its item's matrix W (initially M, symmetric: the
// columns are read as rows), w[c][i] = rows 2i, 2i+1 of column CPL j + c as a packed pair, and their squared
// norms.  A sweep is 8 x (even step, odd step):
//   even: the pairs (0,1), (2,3) .. of the lane;   odd: the pairs (1,2) .. of the lane and the pair (last column of
//   lane j, first column of lane j+1),
// every pair rotated and then swapped in place.  The straddling pair is computed by both lanes (each from the
// other's column, fetched by shuffle) and each keeps its own half of the result; the outer lanes' columns 0 and
// 15 sit the odd step out.  CPL = 4 (8 matrices per warp) costs the fewest instructions per matrix; CPL = 2
// (4 matrices) has the shorter instruction stream per sweep, for a decode step's few freshly filled pages.
// Result: the columns ranked by norm (descending, ties to the lower position); unit eigenvectors of the leading
// min(r, 8) modes to us[item][token][mode] as pairs (u, u) (r > 8: all 16, plain entries, [token][16]), the 16
// eigenvalues to lam_s[item][mode].
template <int CPL>
__device__ __forceinline__ void jacobi_phase(const float *mat, float2 *us, float *lam_s, uint32_t live, int r, int lane) {
  constexpr int LPI = LOCKS_B / CPL;
  const int item = lane / LPI, j = lane % LPI;
  const bool item_live = (live >> item) & 1u;   // lanes of an absent item compute on zeros
  float2 w[CPL][8];
  {
    const float4 *src = reinterpret_cast<const float4 *>(mat + item * LOCKS_B * LOCKS_B + CPL * j * LOCKS_B);
#pragma unroll
    for (int c = 0; c < CPL; ++c)
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const float4 f = item_live ? src[c * 4 + q4] : make_float4(0.f, 0.f, 0.f, 0.f);
        w[c][2 * q4] = make_float2(f.x, f.y);
        w[c][2 * q4 + 1] = make_float2(f.z, f.w);
      }
  }
  __syncwarp();   // every lane holds its columns: the matrices' shared memory may be overwritten from here on
  auto seg_max = [&](float v) {   // maximum over the lanes of the item
#pragma unroll
    for (int o = 1; o < LPI; o <<= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
  };
  // The rotations square matrix entries: bring the matrix to unit scale first (an exact power of two, taken
  // from its largest entry and undone on the eigenvalues), so that keys of any magnitude are handled alike.
  float unscale = 1.f;
  {
    float amax = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c)
#pragma unroll
      for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fmaxf(fabsf(w[c][i].x), fabsf(w[c][i].y)));
    amax = seg_max(amax);
    if (amax > 0.f && amax < INFINITY) {
      int ex;
      (void)frexpf(amax, &ex);
      ex = max(-120, min(120, ex));
      const float sc = ldexpf(1.f, -ex);
      unscale = ldexpf(1.f, ex);
      const float2 sc2 = make_float2(sc, sc);
#pragma unroll
      for (int c = 0; c < CPL; ++c)
#pragma unroll
        for (int i = 0; i < 8; ++i) w[c][i] = mul2(w[c][i], sc2);
    }
  }
  float n[CPL];
  auto norms = [&]() {
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
      float2 acc = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc = fma2(w[c][i], w[c][i], acc);
      n[c] = acc.x + acc.y;
    }
  };
  auto dot = [&](const float2 (&a)[8], const float2 (&b)[8]) {
    float2 acc0 = mul2(a[0], b[0]), acc1 = mul2(a[1], b[1]);
#pragma unroll
    for (int i = 2; i < 8; i += 2) { acc0 = fma2(a[i], b[i], acc0); acc1 = fma2(a[i + 1], b[i + 1], acc1); }
    return (acc0.x + acc1.x) + (acc0.y + acc1.y);
  };
  const float tol2 = LOCKS_BUILD_COS_TOL * LOCKS_BUILD_COS_TOL;
  int bad = 0;
  float floor_n = 0.f;
  // columns whose norm is rounding noise beside the largest (null directions) do not hold up convergence
  auto check = [&](float a, float b, float g) { bad |= (int)(g * g > tol2 * a * b) & (int)(fminf(a, b) > floor_n); };
  // rotate columns P, Q of this lane and swap them
  auto pair_in_lane = [&](float2 (&wp)[8], float2 (&wq)[8], float &np, float &nq) {
    const float g = dot(wp, wq);
    check(np, nq, g);
    float c, sn;
    jacobi_angle(np, nq, g, c, sn);
    const float2 C2 = make_float2(c, c), S2 = make_float2(sn, sn), nS2 = make_float2(-sn, -sn);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 pp = fma2(C2, wp[i], mul2(nS2, wq[i]));
      const float2 qq = fma2(S2, wp[i], mul2(C2, wq[i]));
      wp[i] = qq;
      wq[i] = pp;
    }
    const float cc = c * c, ss = sn * sn, x2 = 2.f * c * sn * g;
    const float na = fmaxf(fmaf(cc, np, fmaf(ss, nq, -x2)), 0.f), nb = fmaxf(fmaf(ss, np, fmaf(cc, nq, x2)), 0.f);
    np = nb;
    nq = na;
  };
  for (int sweep = 0; sweep < LOCKS_BUILD_SWEEPS; ++sweep) {
    norms();
    {
      float nm = n[0];
#pragma unroll
      for (int c = 1; c < CPL; ++c) nm = fmaxf(nm, n[c]);
      floor_n = 1e-11f * seg_max(nm);   // squared norm = squared eigenvalue: modes below 3e-6 of the largest
    }
    bad = 0;
#pragma unroll 1
    for (int st2 = 0; st2 < 8; ++st2) {
#pragma unroll
      for (int c = 0; c + 1 < CPL; c += 2) pair_in_lane(w[c], w[c + 1], n[c], n[c + 1]);
      // odd step: the straddling pairs first (they read the lane's outer columns, which its inner pairs do not touch)
      float2 qr[8], pr[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        qr[i].x = __shfl_down_sync(0xffffffffu, w[0][i].x, 1, LPI);
        qr[i].y = __shfl_down_sync(0xffffffffu, w[0][i].y, 1, LPI);
        pr[i].x = __shfl_up_sync(0xffffffffu, w[CPL - 1][i].x, 1, LPI);
        pr[i].y = __shfl_up_sync(0xffffffffu, w[CPL - 1][i].y, 1, LPI);
      }
      const float nqr = __shfl_down_sync(0xffffffffu, n[0], 1, LPI), npr = __shfl_up_sync(0xffffffffu, n[CPL - 1], 1, LPI);
      // pair A: p = own last column, q = next lane's column 0; this lane's last column becomes q' = s p + c q
      {
        const float g = dot(w[CPL - 1], qr);
        float c, sn;
        jacobi_angle(n[CPL - 1], nqr, g, c, sn);
        check(n[CPL - 1], j == LPI - 1 ? 0.f : nqr, g);   // (the outer lane's pair does not exist: norm 0 never counts)
        c = j == LPI - 1 ? 0.f : c; sn = j == LPI - 1 ? 1.f : sn;
        const float2 C2 = make_float2(c, c), S2 = make_float2(sn, sn);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[CPL - 1][i] = fma2(S2, w[CPL - 1][i], mul2(C2, qr[i]));
        n[CPL - 1] = fmaxf(fmaf(sn * sn, n[CPL - 1], fmaf(c * c, nqr, 2.f * c * sn * g)), 0.f);
      }
      // pair B: p = previous lane's last column, q = own column 0; this lane's column 0 becomes p' = c p - s q
      {
        const float g = dot(pr, w[0]);
        float c, sn;
        jacobi_angle(npr, n[0], g, c, sn);
        c = j == 0 ? 0.f : c; sn = j == 0 ? -1.f : sn;
        const float2 C2 = make_float2(c, c), nS2 = make_float2(-sn, -sn);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[0][i] = fma2(C2, pr[i], mul2(nS2, w[0][i]));
        n[0] = fmaxf(fmaf(c * c, npr, fmaf(sn * sn, n[0], -2.f * c * sn * g)), 0.f);
      }
#pragma unroll
      for (int c = 1; c + 1 < CPL; c += 2) pair_in_lane(w[c], w[c + 1], n[c], n[c + 1]);
    }
    if (!__any_sync(0xffffffffu, bad != 0)) break;
  }
  norms();
  int rank[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) rank[c] = 0;
#pragma unroll
  for (int jj = 0; jj < LPI; ++jj)
#pragma unroll
    for (int cc = 0; cc < CPL; ++cc) {
      const float o = __shfl_sync(0xffffffffu, n[cc], (lane & ~(LPI - 1)) + jj);
#pragma unroll
      for (int c = 0; c < CPL; ++c) rank[c] += (o > n[c]) || (o == n[c] && (jj * CPL + cc) < (j * CPL + c));
    }
#pragma unroll
  for (int c = 0; c < CPL; ++c) {
    lam_s[item * LOCKS_B + rank[c]] = sqrtf(n[c]) * unscale;
    const float inv = n[c] > 0.f ? rsqrtf(n[c]) : 0.f;
    if (r > 8) {   // ranks above 8 (fp32 summaries): all 16 modes, plain entries
      float *dst = reinterpret_cast<float *>(us) + item * LOCKS_B * LOCKS_B + rank[c];
#pragma unroll
      for (int i = 0; i < 8; ++i) { dst[(2 * i) * LOCKS_B] = w[c][i].x * inv; dst[(2 * i + 1) * LOCKS_B] = w[c][i].y * inv; }
    } else if (rank[c] < 8) {
      float2 *dst = us + item * LOCKS_B * 8 + rank[c];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float u0 = w[c][i].x * inv, u1 = w[c][i].y * inv;
        dst[(2 * i) * 8] = make_float2(u0, u0);
        dst[(2 * i + 1) * 8] = make_float2(u1, u1);
      }
    }
  }
  __syncwarp();
}

// The same iteration with one column per lane (16 lanes per matrix, 2 matrices per warp): every pair straddles two
// lanes, so a step is one column fetch, one rotation and half of its result per lane.  Most instructions per
// matrix, shortest instruction stream per sweep: the variant for the page a decode step has just filled, where
// the summary must be ready before the step ends.
__device__ __forceinline__ void jacobi_phase_single(const float *mat, float2 *us, float *lam_s, uint32_t live, int r, int lane) {
  const int item = lane >> 4, j = lane & 15;
  const bool item_live = (live >> item) & 1u;
  float2 w[8];
  {
    const float4 *src = reinterpret_cast<const float4 *>(mat + item * LOCKS_B * LOCKS_B + j * LOCKS_B);
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      const float4 f = item_live ? src[q4] : make_float4(0.f, 0.f, 0.f, 0.f);
      w[2 * q4] = make_float2(f.x, f.y);
      w[2 * q4 + 1] = make_float2(f.z, f.w);
    }
  }
  __syncwarp();
  auto seg_max = [&](float v) {
#pragma unroll
    for (int o = 1; o < 16; o <<= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
  };
  float unscale = 1.f;
  {
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fmaxf(fabsf(w[i].x), fabsf(w[i].y)));
    amax = seg_max(amax);
    if (amax > 0.f && amax < INFINITY) {
      int ex;
      (void)frexpf(amax, &ex);
      ex = max(-120, min(120, ex));
      const float sc = ldexpf(1.f, -ex);
      unscale = ldexpf(1.f, ex);
      const float2 sc2 = make_float2(sc, sc);
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] = mul2(w[i], sc2);
    }
  }
  float n = 0.f;
  auto norm = [&]() {
    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc = fma2(w[i], w[i], acc);
    n = acc.x + acc.y;
  };
  const float tol2 = LOCKS_BUILD_COS_TOL * LOCKS_BUILD_COS_TOL;
  for (int sweep = 0; sweep < LOCKS_BUILD_SWEEPS; ++sweep) {
    norm();
    const float floor_n = 1e-11f * seg_max(n);
    int bad = 0;
#pragma unroll 1
    for (int step = 0; step < LOCKS_B; ++step) {
      // even step: pairs (2m, 2m+1); odd step: pairs (2m+1, 2m+2), lanes 0 and 15 idle.  The lower position is p.
      const int odd = step & 1;
      const bool is_p = ((j ^ odd) & 1) == 0;
      const bool idle = odd && (j == 0 || j == 15);
      const int partner = (lane & 16) + (is_p ? min(j + 1, 15) : max(j - 1, 0));
      float2 o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        o[i].x = __shfl_sync(0xffffffffu, w[i].x, partner);
        o[i].y = __shfl_sync(0xffffffffu, w[i].y, partner);
      }
      const float no = __shfl_sync(0xffffffffu, n, partner);
      float2 acc0 = mul2(w[0], o[0]), acc1 = mul2(w[1], o[1]);
#pragma unroll
      for (int i = 2; i < 8; i += 2) { acc0 = fma2(w[i], o[i], acc0); acc1 = fma2(w[i + 1], o[i + 1], acc1); }
      const float g = (acc0.x + acc1.x) + (acc0.y + acc1.y);
      const float a = is_p ? n : no, b = is_p ? no : n;   // |p|^2, |q|^2
      bad |= (int)(!idle) & (int)(g * g > tol2 * a * b) & (int)(fminf(a, b) > floor_n);
      float c, sn;
      jacobi_angle(a, b, g, c, sn);
      // rotate and swap: the lane that held p now holds q' = s p + c q, the lane that held q holds p' = c p - s q
      float ca = is_p ? sn : -sn, cb = c;   // new = ca * own + cb * other
      float nn = is_p ? fmaf(sn * sn, a, fmaf(c * c, b, 2.f * c * sn * g)) : fmaf(c * c, a, fmaf(sn * sn, b, -2.f * c * sn * g));
      if (idle) { ca = 1.f; cb = 0.f; nn = n; }
      const float2 A2 = make_float2(ca, ca), B2 = make_float2(cb, cb);
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] = fma2(A2, w[i], mul2(B2, o[i]));
      n = fmaxf(nn, 0.f);
    }
    if (!__any_sync(0xffffffffu, bad != 0)) break;
  }
  norm();
  int rank = 0;
#pragma unroll
  for (int jj = 0; jj < 16; ++jj) {
    const float o = __shfl_sync(0xffffffffu, n, (lane & 16) + jj);
    rank += (o > n) || (o == n && jj < j);
  }
  lam_s[item * LOCKS_B + rank] = sqrtf(n) * unscale;
  const float inv = n > 0.f ? rsqrtf(n) : 0.f;
  if (r > 8) {
    float *dst = reinterpret_cast<float *>(us) + item * LOCKS_B * LOCKS_B + rank;
#pragma unroll
    for (int i = 0; i < 8; ++i) { dst[(2 * i) * LOCKS_B] = w[i].x * inv; dst[(2 * i + 1) * LOCKS_B] = w[i].y * inv; }
  } else if (rank < 8) {
    float2 *dst = us + item * LOCKS_B * 8 + rank;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float u0 = w[i].x * inv, u1 = w[i].y * inv;
      dst[(2 * i) * 8] = make_float2(u0, u0);
      dst[(2 * i + 1) * 8] = make_float2(u1, u1);
    }
  }
  __syncwarp();
}

// STEP: the launch inside a decode step (one freshly filled page per warp at most); otherwise the bulk build.
template <typename T, int FMT, bool STEP>
__global__ void __launch_bounds__(kBuildWarps * 32, kBuildCtasPerSm) build_kernel(BuildParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (STEP && p.hint && blockIdx.x == 0 && warp == 0)
    locks_update_partition_hint(p.hint, p.seq_lens, p.batch, p.Hkv, p.kpages, p.hint_wpp, p.hint_rounds, p.hint_W, lane);
  // ---- the warp's items: lane s < 8 works out item s
  // (a decode step gives every page that just filled a warp of its own: there the latency counts, not the throughput)
  int it_b = 0, it_h = 0, it_block = -1, it_new = 0;
  constexpr int ipw = STEP ? 1 : kBuildItems;
  if (lane < ipw) {
    int page = -1;
    const int slot = (blockIdx.x * kBuildWarps + warp) * ipw + lane;
    if (STEP) {
      if (slot < p.batch * p.Hkv) {
        it_b = slot / p.Hkv; it_h = slot - it_b * p.Hkv;
        const int Tb = p.seq_lens[it_b];
        if (Tb > 0 && (Tb % LOCKS_B) == 0) {
          page = Tb / LOCKS_B - 1;
          it_new = (p.k_new && p.append_pos && p.append_pos[it_b] == Tb - 1) ? 1 : 0;   // row 15 is this step's token
        }
      }
    } else {
      it_b = blockIdx.z % p.batch; it_h = blockIdx.y;
      const int complete = p.seq_lens[it_b] / LOCKS_B;
      const int p0 = p.page_begin ? p.page_begin[it_b] : 0;
      const int p1 = min(p.page_end ? p.page_end[it_b] : complete, complete);
      page = p0 + slot;
      if (page < 0 || page >= p1) page = -1;
    }
    if (page >= p.Pmax) page = -1;
    if (page >= 0) {
      it_block = p.block_table[(int64_t)it_b * p.Pmax + page];
      if (it_block < 0 || it_block >= p.num_blocks) {
        set_status(p.status, LOCKS_ERR_BAD_BLOCK);
        it_block = -1;
      }
    }
  }
  const uint32_t live = __ballot_sync(0xffffffffu, it_block >= 0);
  if (!live) return;

  const int layer = STEP ? 0 : blockIdx.z / p.batch;
  const void *kbase = p.k_layers ? p.k_layers[layer] : p.k;
  uint8_t *sbase = p.summ_layers ? reinterpret_cast<uint8_t *>(p.summ_layers[layer]) : p.summ;
  uint8_t *scratch = smem_raw + warp * kBuildSmemPerWarp;                        // D half-tiles; phase 3: the blob
  float *mat = reinterpret_cast<float *>(scratch + kBuildScratch);              // [8][16][16] Gram; then [8][16][8] pairs (u, u) of U_r
  float *kn_s = mat + kBuildItems * LOCKS_B * LOCKS_B;                          // [8] squared norm of the page's keys
  float *lam_s = kn_s + 16;                                                     // [8][16] eigenvalues, descending
  float2 *us = reinterpret_cast<float2 *>(mat);
  const int r = p.r;

  // keys of item s: v[i][c] = key i, dim 4 lane + c, as fp32
  auto load_item = [&](int s, float (&v)[LOCKS_B][4]) {
    const int b = __shfl_sync(0xffffffffu, it_b, s), h = __shfl_sync(0xffffffffu, it_h, s);
    const int block = __shfl_sync(0xffffffffu, it_block, s), nw = __shfl_sync(0xffffffffu, it_new, s);
    const T *K = reinterpret_cast<const T *>(kbase) + ((int64_t)block * p.sb + (int64_t)h * p.sh) + 4 * lane;
    const T *Knew = reinterpret_cast<const T *>(p.k_new) + ((int64_t)b * p.Hkv + h) * LOCKS_D + 4 * lane;
#pragma unroll
    for (int i = 0; i < LOCKS_B; ++i) {
      const T *src = (i == LOCKS_B - 1 && nw) ? Knew : K + (int64_t)i * p.st;
      if (sizeof(T) == 2) {
        const uint2 w = *reinterpret_cast<const uint2 *>(src);
        v[i][0] = __uint_as_float(w.x << 16); v[i][1] = __uint_as_float(w.x & 0xFFFF0000u);
        v[i][2] = __uint_as_float(w.y << 16); v[i][3] = __uint_as_float(w.y & 0xFFFF0000u);
      } else {
        const float4 w = *reinterpret_cast<const float4 *>(src);
        v[i][0] = w.x; v[i][1] = w.y; v[i][2] = w.z; v[i][3] = w.w;
      }
    }
  };
  auto centre = [&](float (&v)[LOCKS_B][4], float (&mu)[4]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) mu[c] = 0.f;
#pragma unroll
    for (int i = 0; i < LOCKS_B; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) mu[c] += v[i][c];
#pragma unroll
    for (int c = 0; c < 4; ++c) mu[c] *= (1.f / LOCKS_B);
#pragma unroll
    for (int i = 0; i < LOCKS_B; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) v[i][c] -= mu[c];
  };

  // ---- 1. Gram matrices M = D D^T on the tensor cores.  D = H + L with H = bf16(D), L = bf16(D - H) (16 significant
  // bits; the bf16 products are exact and accumulate in fp32): M = (H H^T + L L^T) + H L^T + (H L^T)^T.  The A
  // operand (tokens x dims) and the B operand (dims x tokens) of an m16n8k16 step are the same registers.
  // Two passes over 64 dims each: the half-tiles of H and L (16 rows x 128 bytes, 16-byte chunks XOR-swizzled with
  // the row so that ldmatrix reads are conflict-free) share the 4 KB of scratch; in a pass the 16 lanes that own
  // the half's dims write it.
#pragma unroll 1
  for (int s = 0; s < kBuildItems; ++s) {
    if (!((live >> s) & 1u)) continue;
    uint32_t hl[LOCKS_B][4];   // h01, h23, l01, l23 of this lane's 4 dims, per key
    {
      float v[LOCKS_B][4], mu[4];
      load_item(s, v);
      float knorm2 = 0.f;
#pragma unroll
      for (int i = 0; i < LOCKS_B; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) knorm2 = fmaf(v[i][c], v[i][c], knorm2);
      knorm2 = warp_sum(knorm2);
      if (lane == 0) kn_s[s] = knorm2;
      centre(v, mu);
#pragma unroll
      for (int i = 0; i < LOCKS_B; ++i) {
        const uint32_t h01 = pack_bf16(v[i][0], v[i][1]), h23 = pack_bf16(v[i][2], v[i][3]);
        hl[i][0] = h01; hl[i][1] = h23;
        hl[i][2] = pack_bf16(v[i][0] - __uint_as_float(h01 << 16), v[i][1] - __uint_as_float(h01 & 0xFFFF0000u));
        hl[i][3] = pack_bf16(v[i][2] - __uint_as_float(h23 << 16), v[i][3] - __uint_as_float(h23 & 0xFFFF0000u));
      }
    }
    float X0[4] = {0.f, 0.f, 0.f, 0.f}, X1[4] = {0.f, 0.f, 0.f, 0.f}, Y0[4] = {0.f, 0.f, 0.f, 0.f}, Y1[4] = {0.f, 0.f, 0.f, 0.f};
    const int c16 = lane & 15;                                          // writer: dims 4 c16 .. + 3 of the half
    const int mq = lane >> 3, rr = lane & 7, tok = (mq & 1) * 8 + rr;   // reader (ldmatrix address lanes)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      if ((lane >> 4) == hf) {
#pragma unroll
        for (int row = 0; row < LOCKS_B; ++row) {
          uint8_t *dst = scratch + row * 128 + ((((c16 >> 1) ^ (row & 7)) << 4) | ((c16 & 1) << 3));
          *reinterpret_cast<uint2 *>(dst) = make_uint2(hl[row][0], hl[row][1]);
          *reinterpret_cast<uint2 *>(dst + 2048) = make_uint2(hl[row][2], hl[row][3]);
        }
      }
      __syncwarp();
#pragma unroll
      for (int s4 = 0; s4 < 4; ++s4) {
        uint32_t Hf[4], Lf[4];
        const uint8_t *src = scratch + tok * 128 + (((2 * s4 + (mq >> 1)) ^ (tok & 7)) << 4);
        ldsm_x4(Hf, src);
        ldsm_x4(Lf, src + 2048);
        mma_bf16(X0, Hf[0], Hf[1], Hf[2], Hf[3], Hf[0], Hf[2]);
        mma_bf16(X1, Hf[0], Hf[1], Hf[2], Hf[3], Hf[1], Hf[3]);
        mma_bf16(X0, Lf[0], Lf[1], Lf[2], Lf[3], Lf[0], Lf[2]);
        mma_bf16(X1, Lf[0], Lf[1], Lf[2], Lf[3], Lf[1], Lf[3]);
        mma_bf16(Y0, Hf[0], Hf[1], Hf[2], Hf[3], Lf[0], Lf[2]);
        mma_bf16(Y1, Hf[0], Hf[1], Hf[2], Hf[3], Lf[1], Lf[3]);
      }
      __syncwarp();
    }
    // accumulator (x = lane / 4, t = lane % 4): [0..1] = row x, columns 2t, 2t+1; [2..3] = row x + 8.
    // M = sym(X) + Y + Y^T, assembled through two padded 16 x 17 arrays in the (now free) scratch
    {
      float *XA = reinterpret_cast<float *>(scratch), *YA = XA + LOCKS_B * 17;
      const int x = lane >> 2, t = lane & 3;
      XA[x * 17 + 2 * t] = X0[0]; XA[x * 17 + 2 * t + 1] = X0[1]; XA[(x + 8) * 17 + 2 * t] = X0[2]; XA[(x + 8) * 17 + 2 * t + 1] = X0[3];
      XA[x * 17 + 8 + 2 * t] = X1[0]; XA[x * 17 + 9 + 2 * t] = X1[1]; XA[(x + 8) * 17 + 8 + 2 * t] = X1[2]; XA[(x + 8) * 17 + 9 + 2 * t] = X1[3];
      YA[x * 17 + 2 * t] = Y0[0]; YA[x * 17 + 2 * t + 1] = Y0[1]; YA[(x + 8) * 17 + 2 * t] = Y0[2]; YA[(x + 8) * 17 + 2 * t + 1] = Y0[3];
      YA[x * 17 + 8 + 2 * t] = Y1[0]; YA[x * 17 + 9 + 2 * t] = Y1[1]; YA[(x + 8) * 17 + 8 + 2 * t] = Y1[2]; YA[(x + 8) * 17 + 9 + 2 * t] = Y1[3];
      __syncwarp();
      const int i = lane >> 1, j0 = 8 * (lane & 1);
      float g[8];
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        const int j = j0 + jj;
        g[jj] = 0.5f * (XA[i * 17 + j] + XA[j * 17 + i]) + YA[i * 17 + j] + YA[j * 17 + i];
      }
      float4 *dst = reinterpret_cast<float4 *>(mat + s * LOCKS_B * LOCKS_B + i * LOCKS_B + j0);
      dst[0] = make_float4(g[0], g[1], g[2], g[3]);
      dst[1] = make_float4(g[4], g[5], g[6], g[7]);
      __syncwarp();
    }
  }

  // ---- 2. eigenvectors and eigenvalues of all the warp's items at once
  if (STEP) jacobi_phase_single(mat, us, lam_s, live, r, lane);
  else jacobi_phase<4>(mat, us, lam_s, live, r, lane);

  // ---- 3. per item: modes, basis, coefficients, quantisation
  uint8_t *blob = scratch;
#pragma unroll 1
  for (int s = 0; s < kBuildItems; ++s) {
    if (!((live >> s) & 1u)) continue;
    float dv[LOCKS_B][4], mu[4];
    load_item(s, dv);
    centre(dv, mu);
    const int block = __shfl_sync(0xffffffffu, it_block, s), h = __shfl_sync(0xffffffffu, it_h, s);
    const float knorm2 = kn_s[s];
    const float2 *U = us + s * LOCKS_B * 8;      // [token][mode], (u, u); ranks above 8: Uw[token][16 modes]
    const float *Uw = reinterpret_cast<const float *>(us) + s * LOCKS_B * LOCKS_B;
    const float *lamv = lam_s + s * LOCKS_B;     // eigenvalues, descending
    // ---- choose r_eff
    const float lam0 = lamv[0];
    int r_eff = 0;
    const int rmax = min(r, LOCKS_B - 1);
    for (int l = 0; l < rmax; ++l) {
      const float ll = lamv[l];
      if (lam0 > 0.f && ll > 1e-6f * lam0 && ll > 1e-10f * knorm2) r_eff = l + 1; else break;
    }
    // ---- per mode: basis entries of this lane's 4 dims, sign, quantise
    if (FMT == LOCKS_FMT_I4) {
      for (int e = lane; e < i4_stride(8) / 4; e += 32) reinterpret_cast<uint32_t *>(blob)[e] = 0u;
      __syncwarp();
    }
    uint8_t *gout = sbase + ((int64_t)block * p.Hkv + h) * p.S;
    float *fout = reinterpret_cast<float *>(gout);
    uint32_t sign_bits = 0u;   // bit l: mode l was flipped
#pragma unroll 1
    for (int l = 0; l < r; ++l) {
      float v[4] = {0.f, 0.f, 0.f, 0.f};
      float best = 0.f;   // largest magnitude of the mode's basis vector
      if (l < r_eff) {
        const float inv = rsqrtf(lamv[l]);
        float2 va = make_float2(0.f, 0.f), vb = make_float2(0.f, 0.f);
        if (r > 8) {
#pragma unroll
          for (int i = 0; i < LOCKS_B; ++i) {
            const float u1 = Uw[i * LOCKS_B + l];
            const float2 u = make_float2(u1, u1);
            va = fma2(make_float2(dv[i][0], dv[i][1]), u, va);
            vb = fma2(make_float2(dv[i][2], dv[i][3]), u, vb);
          }
        } else {
#pragma unroll
          for (int i = 0; i < LOCKS_B; ++i) {
            const float2 u = U[i * 8 + l];
            va = fma2(make_float2(dv[i][0], dv[i][1]), u, va);
            vb = fma2(make_float2(dv[i][2], dv[i][3]), u, vb);
          }
        }
        v[0] = va.x * inv; v[1] = va.y * inv; v[2] = vb.x * inv; v[3] = vb.y * inv;
        // sign: entry of largest magnitude (lowest dim on ties) positive.  Magnitudes order like their bit
        // patterns; the lowest lane that holds the maximum owns the lowest such dim.
        best = fabsf(v[0]); float bv = v[0];
#pragma unroll
        for (int c = 1; c < 4; ++c) if (fabsf(v[c]) > best) { best = fabsf(v[c]); bv = v[c]; }
        const uint32_t mxb = __reduce_max_sync(0xffffffffu, __float_as_uint(best));
        const uint32_t who = __ballot_sync(0xffffffffu, __float_as_uint(best) == mxb);
        bv = __shfl_sync(0xffffffffu, bv, __ffs(who) - 1);
        best = __uint_as_float(mxb);
        if (bv < 0.f) {
          sign_bits |= 1u << l;
#pragma unroll
          for (int c = 0; c < 4; ++c) v[c] = -v[c];
        }
      }
      if (FMT == LOCKS_FMT_F32) {
        *reinterpret_cast<float4 *>(fout + LOCKS_D + l * LOCKS_D + lane * 4) = make_float4(v[0], v[1], v[2], v[3]);
      } else if (FMT == LOCKS_FMT_BF16) {   // row-major bf16 basis, straight to global memory
        *reinterpret_cast<uint2 *>(gout + 2 * (l * LOCKS_D + lane * 4)) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
      } else if (FMT == LOCKS_FMT_I8) {     // row-major int8 basis, one scale per mode
        const __half sh = __float2half_rn(best / 127.f);
        const float sc = inv_scale(__half2float(sh));
        if (lane == 0) *reinterpret_cast<__half *>(gout + wb_off_sv(r, 1) + 2 * l) = sh;
        uint32_t wd = 0u;
#pragma unroll
        for (int c = 0; c < 4; ++c) wd |= (uint32_t)((int)round_code(v[c], sc, 127.f) + 128) << (8 * c);
        *reinterpret_cast<uint32_t *>(gout + l * LOCKS_D + lane * 4) = wd;
      } else {
        const __half sh = __float2half_rn(best / 7.f);
        const float sc = inv_scale(__half2float(sh));
        if (lane == 0) *reinterpret_cast<__half *>(blob + i4_off_sv(r) + 2 * l) = sh;
        // lane = 8 t + s8 owns dims 32 t + 4 s8 + {0,1,2,3} = (half, e) in {0,1}^2 of k-step s8
        const int t = lane >> 3, s8 = lane & 7, i0 = (s8 & 1) << 1;
        uint32_t nb[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) nb[c] = (uint32_t)((int)round_code(v[c], sc, 7.f) + 8);
        // dim offset c = 2*half + e -> nibble i0 + half + 4 e
        uint32_t pw = (nb[0] << (4 * i0)) | (nb[1] << (4 * (i0 + 4))) | (nb[2] << (4 * (i0 + 1))) | (nb[3] << (4 * (i0 + 5)));
        pw |= __shfl_xor_sync(0xffffffffu, pw, 1);
        if ((s8 & 1) == 0) *reinterpret_cast<uint32_t *>(blob + (l * 4 + t) * 16 + (s8 >> 1) * 4) = pw;
      }
    }
    // coefficients: lane i < 16 owns token i
    if (lane < LOCKS_B) {
      float cf[16];
      float mx = 0.f;
      for (int l = 0; l < r; ++l) {
        float c = 0.f;
        if (l < r_eff) {
          c = sqrtf(lamv[l]) * (r > 8 ? Uw[lane * LOCKS_B + l] : U[lane * 8 + l].x);
          if ((sign_bits >> l) & 1u) c = -c;
        }
        cf[l & 15] = c;
        mx = fmaxf(mx, fabsf(c));
      }
      if (FMT == LOCKS_FMT_F32) {
        for (int l = 0; l < r; ++l) fout[LOCKS_D + r * LOCKS_D + lane * r + l] = cf[l & 15];
      } else if (FMT == LOCKS_FMT_I8 || FMT == LOCKS_FMT_BF16) {
        constexpr int W = FMT == LOCKS_FMT_BF16 ? 2 : 1;
        const __half sh = __float2half_rn(mx / 127.f);
        const float sc = inv_scale(__half2float(sh));
        *reinterpret_cast<__half *>(gout + wb_off_sc(r, W) + 2 * lane) = sh;
        for (int l = 0; l < r; ++l) gout[wb_off_coef(r, W) + lane * r + l] = (uint8_t)((int)round_code(cf[l & 15], sc, 127.f) + 128);
      } else {
        const __half sh = __float2half_rn(mx / 127.f);
        const float sc = inv_scale(__half2float(sh));
        const int tpos = ((lane & 7) >> 1) * 4 + (lane >> 3) * 2 + (lane & 1);
        *reinterpret_cast<__half *>(blob + i4_off_sc(r) + 2 * tpos) = sh;
        const int xx = lane & 7, hi = lane >> 3;
        for (int l = 0; l < r; ++l)
          blob[i4_off_coef(r) + (xx * (r / 2) + (l >> 1)) * 4 + hi * 2 + (l & 1)] =
              (uint8_t)((int)round_code(cf[l & 15], sc, 127.f) + 128);
      }
    }
    // centroid
    if (FMT == LOCKS_FMT_F32) {
      *reinterpret_cast<float4 *>(fout + lane * 4) = make_float4(mu[0], mu[1], mu[2], mu[3]);
    } else if (FMT == LOCKS_FMT_I8 || FMT == LOCKS_FMT_BF16) {
      constexpr int W = FMT == LOCKS_FMT_BF16 ? 2 : 1;
      float mx = fmaxf(fmaxf(fabsf(mu[0]), fabsf(mu[1])), fmaxf(fabsf(mu[2]), fabsf(mu[3])));
      mx = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
      const __half sh = __float2half_rn(mx / 127.f);
      const float sc = inv_scale(__half2float(sh));
      if (lane == 0) *reinterpret_cast<__half *>(gout + wb_off_smu(r, W)) = sh;
      uint32_t wd = 0u;
#pragma unroll
      for (int c = 0; c < 4; ++c) wd |= (uint32_t)((int)round_code(mu[c], sc, 127.f) + 128) << (8 * c);
      *reinterpret_cast<uint32_t *>(gout + wb_off_mu(r, W) + lane * 4) = wd;
      // bytes between the payload and the 16-byte padded stride stay zero (the buffer is the caller's; clear them)
      for (int e = wb_off_smu(r, W) + 2 + lane; e < p.S; e += 32) gout[e] = 0;
    } else {
      float mx = fmaxf(fmaxf(fabsf(mu[0]), fabsf(mu[1])), fmaxf(fabsf(mu[2]), fabsf(mu[3])));
      mx = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
      const __half sh = __float2half_rn(mx / 127.f);
      const float sc = inv_scale(__half2float(sh));
      if (lane == 0) *reinterpret_cast<__half *>(blob + i4_off_smu(r)) = sh;
      uint32_t bytes[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) bytes[c] = (uint32_t)((int)round_code(mu[c], sc, 127.f) + 128);
      // dim offset c = 2*half + e -> byte e*2 + half
      const uint32_t wd = bytes[0] | (bytes[2] << 8) | (bytes[1] << 16) | (bytes[3] << 24);
      *reinterpret_cast<uint32_t *>(blob + i4_off_mu(r) + lane * 4) = wd;
      __syncwarp();
      uint4 *dst = reinterpret_cast<uint4 *>(gout);
      for (int e = lane; e < p.S / 16; e += 32) dst[e] = reinterpret_cast<const uint4 *>(blob)[e];
      __syncwarp();   // the blob is cleared again for the next item
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Pages of 32 and 64 tokens (App. D "Page size"): one warp per (page, KV head), everything in fp32 from shared
// memory, the row-major summary formats only.  The same method as above (centre, Gram, one-sided Jacobi by
// odd-even transposition, rank, project, quantise), written for brevity rather than speed: lane m rotates the
// column pair m of a step.
// ------------------------------------------------------------------------------------------------
constexpr int kWideDStride = LOCKS_D + 4;   // floats per staged key row (16-byte aligned rows, no bank conflicts)
__host__ __device__ constexpr int build_wide_smem(int B) {
  return (B * kWideDStride + B * (B + 1) + 2 * B + 32) * 4;   // keys, W (column-major, padded), norms, order, misc
}

template <typename T, int FMT>
__global__ void __launch_bounds__(32) build_wide_kernel(BuildParams p, int B, int step) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int lane = threadIdx.x;
  int b, h, page, last_from_new = 0;
  if (step) {
    const int prob = blockIdx.x;
    if (prob >= p.batch * p.Hkv) return;
    b = prob / p.Hkv; h = prob - b * p.Hkv;
    const int Tb = p.seq_lens[b];
    if (Tb <= 0 || (Tb % B) != 0) return;
    page = Tb / B - 1;
    last_from_new = (p.k_new && p.append_pos && p.append_pos[b] == Tb - 1) ? 1 : 0;
  } else {
    b = blockIdx.z; h = blockIdx.y;
    const int complete = p.seq_lens[b] / B;
    const int p0 = p.page_begin ? p.page_begin[b] : 0;
    const int p1 = min(p.page_end ? p.page_end[b] : complete, complete);
    page = p0 + blockIdx.x;
    if (page < 0 || page >= p1) return;
  }
  if (page >= p.Pmax) return;
  const int block = p.block_table[(int64_t)b * p.Pmax + page];
  if (block < 0 || block >= p.num_blocks) {
    if (lane == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
    return;
  }
  float *Ds = reinterpret_cast<float *>(smem_raw);   // [B][kWideDStride] deviations
  float *W = Ds + B * kWideDStride;                  // [B columns][B + 1]
  float *nr = W + B * (B + 1);                       // [B] squared column norms
  int *order = reinterpret_cast<int *>(nr + B);      // [B] column of rank l
  const int WS = B + 1, r = p.r;
  // ---- keys, centroid, deviations
  float mu[4] = {0.f, 0.f, 0.f, 0.f}, knorm2 = 0.f;
  {
    const T *K = reinterpret_cast<const T *>(p.k) + ((int64_t)block * p.sb + (int64_t)h * p.sh) + 4 * lane;
    const T *Knew = reinterpret_cast<const T *>(p.k_new) + ((int64_t)b * p.Hkv + h) * LOCKS_D + 4 * lane;
    for (int i = 0; i < B; ++i) {
      const T *src = (i == B - 1 && last_from_new) ? Knew : K + (int64_t)i * p.st;
      float v[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] = ldf<T>(src, c);
#pragma unroll
      for (int c = 0; c < 4; ++c) { mu[c] += v[c]; knorm2 = fmaf(v[c], v[c], knorm2); }
      *reinterpret_cast<float4 *>(Ds + i * kWideDStride + 4 * lane) = make_float4(v[0], v[1], v[2], v[3]);
    }
    knorm2 = warp_sum(knorm2);
#pragma unroll
    for (int c = 0; c < 4; ++c) mu[c] /= (float)B;
    for (int i = 0; i < B; ++i) {
      float4 *d4 = reinterpret_cast<float4 *>(Ds + i * kWideDStride + 4 * lane);
      float4 v = *d4;
      v.x -= mu[0]; v.y -= mu[1]; v.z -= mu[2]; v.w -= mu[3];
      *d4 = v;
    }
    __syncwarp();
  }
  // ---- Gram matrix: lane j (and j + 32) computes column j of M, row by row
  float amax = 0.f;
  for (int jj = lane; jj < B; jj += 32) {
    for (int i = 0; i < B; ++i) {
      const float4 *di = reinterpret_cast<const float4 *>(Ds + i * kWideDStride);
      const float4 *dj = reinterpret_cast<const float4 *>(Ds + jj * kWideDStride);
      float acc = 0.f;
#pragma unroll 8
      for (int c = 0; c < LOCKS_D / 4; ++c) {
        const float4 x = di[c], y = dj[c];
        acc = fmaf(x.x, y.x, fmaf(x.y, y.y, fmaf(x.z, y.z, fmaf(x.w, y.w, acc))));
      }
      W[jj * WS + i] = acc;
      amax = fmaxf(amax, fabsf(acc));
    }
  }
  amax = warp_max(amax);
  // unit scale (an exact power of two, undone on the eigenvalues)
  float unscale = 1.f;
  if (amax > 0.f && amax < INFINITY) {
    int ex;
    (void)frexpf(amax, &ex);
    ex = max(-120, min(120, ex));
    const float sc = ldexpf(1.f, -ex);
    unscale = ldexpf(1.f, ex);
    for (int jj = lane; jj < B; jj += 32)
      for (int i = 0; i < B; ++i) W[jj * WS + i] *= sc;
  }
  __syncwarp();
  // ---- one-sided Jacobi, odd-even transposition, rotate then swap
  const float tol2 = LOCKS_BUILD_COS_TOL * LOCKS_BUILD_COS_TOL;
  for (int sweep = 0; sweep < 2 * LOCKS_BUILD_SWEEPS; ++sweep) {
    float nm = 0.f;
    for (int jj = lane; jj < B; jj += 32) {
      float a = 0.f;
      for (int i = 0; i < B; ++i) a = fmaf(W[jj * WS + i], W[jj * WS + i], a);
      nr[jj] = a;
      nm = fmaxf(nm, a);
    }
    const float floor_n = 1e-11f * warp_max(nm);
    __syncwarp();
    int bad = 0;
    for (int st = 0; st < B; ++st) {
      const int pc = 2 * lane + (st & 1), qc = pc + 1;   // the pair of this lane
      if (qc < B) {
        float *wp = W + pc * WS, *wq = W + qc * WS;
        const float a = nr[pc], bq = nr[qc];
        float g = 0.f;
        for (int i = 0; i < B; ++i) g = fmaf(wp[i], wq[i], g);
        bad |= (int)(g * g > tol2 * a * bq) & (int)(fminf(a, bq) > floor_n);
        float c, sn;
        jacobi_angle(a, bq, g, c, sn);
        for (int i = 0; i < B; ++i) {
          const float x = wp[i], y = wq[i];
          wp[i] = fmaf(sn, x, c * y);    // q' takes p's place
          wq[i] = fmaf(c, x, -sn * y);   // p' takes q's place
        }
        nr[pc] = fmaxf(fmaf(sn * sn, a, fmaf(c * c, bq, 2.f * c * sn * g)), 0.f);
        nr[qc] = fmaxf(fmaf(c * c, a, fmaf(sn * sn, bq, -2.f * c * sn * g)), 0.f);
      }
      __syncwarp();
    }
    if (!__any_sync(0xffffffffu, bad != 0)) break;
  }
  // ---- exact norms, ranking (descending, ties to the lower position)
  for (int jj = lane; jj < B; jj += 32) {
    float a = 0.f;
    for (int i = 0; i < B; ++i) a = fmaf(W[jj * WS + i], W[jj * WS + i], a);
    nr[jj] = a;
  }
  __syncwarp();
  for (int jj = lane; jj < B; jj += 32) {
    const float mine = nr[jj];
    int rk = 0;
    for (int o = 0; o < B; ++o) rk += (nr[o] > mine) || (nr[o] == mine && o < jj);
    order[rk] = jj;
  }
  __syncwarp();
  const float lam0 = sqrtf(nr[order[0]]) * unscale;
  int r_eff = 0;
  const int rmax = min(r, B - 1);
  for (int l = 0; l < rmax; ++l) {
    const float ll = sqrtf(nr[order[l]]) * unscale;
    if (lam0 > 0.f && ll > 1e-6f * lam0 && ll > 1e-10f * knorm2) r_eff = l + 1; else break;
  }
  uint8_t *gout = p.summ + ((int64_t)block * p.Hkv + h) * p.S;
  float *fout = reinterpret_cast<float *>(gout);
  constexpr int WD = FMT == LOCKS_FMT_BF16 ? 2 : 1;
  uint32_t sign_bits = 0u;
  for (int l = 0; l < r; ++l) {
    float v[4] = {0.f, 0.f, 0.f, 0.f}, best = 0.f;
    if (l < r_eff) {
      const int col = order[l];
      const float n2 = nr[col], lam = sqrtf(n2) * unscale;
      const float inv = rsqrtf(n2) * rsqrtf(lam);   // unit eigenvector entries, then 1 / sigma
      for (int i = 0; i < B; ++i) {
        const float u = W[col * WS + i];
        const float4 d4 = *reinterpret_cast<const float4 *>(Ds + i * kWideDStride + 4 * lane);
        v[0] = fmaf(d4.x, u, v[0]); v[1] = fmaf(d4.y, u, v[1]); v[2] = fmaf(d4.z, u, v[2]); v[3] = fmaf(d4.w, u, v[3]);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] *= inv;
      best = fabsf(v[0]); float bv = v[0];
#pragma unroll
      for (int c = 1; c < 4; ++c) if (fabsf(v[c]) > best) { best = fabsf(v[c]); bv = v[c]; }
      const uint32_t mxb = __reduce_max_sync(0xffffffffu, __float_as_uint(best));
      const uint32_t who = __ballot_sync(0xffffffffu, __float_as_uint(best) == mxb);
      bv = __shfl_sync(0xffffffffu, bv, __ffs(who) - 1);
      best = __uint_as_float(mxb);
      if (bv < 0.f) {
        sign_bits |= 1u << l;
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] = -v[c];
      }
    }
    if (FMT == LOCKS_FMT_F32) {
      *reinterpret_cast<float4 *>(fout + LOCKS_D + l * LOCKS_D + lane * 4) = make_float4(v[0], v[1], v[2], v[3]);
    } else if (FMT == LOCKS_FMT_BF16) {
      *reinterpret_cast<uint2 *>(gout + 2 * (l * LOCKS_D + lane * 4)) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
    } else if (FMT == LOCKS_FMT_I8) {
      const __half sh = __float2half_rn(best / 127.f);
      const float sc = inv_scale(__half2float(sh));
      if (lane == 0) *reinterpret_cast<__half *>(gout + wb_off_sv(r, 1, B) + 2 * l) = sh;
      uint32_t wd = 0u;
#pragma unroll
      for (int c = 0; c < 4; ++c) wd |= (uint32_t)((int)round_code(v[c], sc, 127.f) + 128) << (8 * c);
      *reinterpret_cast<uint32_t *>(gout + l * LOCKS_D + lane * 4) = wd;
    } else {   // int4 basis: the same nibble order as at B = 16
      const __half sh = __float2half_rn(best / 7.f);
      const float sc = inv_scale(__half2float(sh));
      if (lane == 0) *reinterpret_cast<__half *>(gout + i4_off_sv(r, B) + 2 * l) = sh;
      const int t = lane >> 3, s8 = lane & 7, i0 = (s8 & 1) << 1;
      uint32_t nb[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) nb[c] = (uint32_t)((int)round_code(v[c], sc, 7.f) + 8);
      uint32_t pw = (nb[0] << (4 * i0)) | (nb[1] << (4 * (i0 + 4))) | (nb[2] << (4 * (i0 + 1))) | (nb[3] << (4 * (i0 + 5)));
      pw |= __shfl_xor_sync(0xffffffffu, pw, 1);
      if ((s8 & 1) == 0) *reinterpret_cast<uint32_t *>(gout + (l * 4 + t) * 16 + (s8 >> 1) * 4) = pw;
    }
  }
  // coefficients: lane owns tokens lane and lane + 32
  for (int tok = lane; tok < B; tok += 32) {
    float mx = 0.f;
    for (int l = 0; l < r; ++l) {
      float c = 0.f;
      if (l < r_eff) {
        const int col = order[l];
        c = W[col * WS + tok] * rsqrtf(nr[col]) * sqrtf(sqrtf(nr[col]) * unscale);
        if ((sign_bits >> l) & 1u) c = -c;
      }
      mx = fmaxf(mx, fabsf(c));
      if (FMT == LOCKS_FMT_F32) fout[LOCKS_D + r * LOCKS_D + tok * r + l] = c;
    }
    if (FMT != LOCKS_FMT_F32) {
      const __half sh = __float2half_rn(mx / 127.f);
      const float sc = inv_scale(__half2float(sh));
      *reinterpret_cast<__half *>(gout + (FMT == LOCKS_FMT_I4 ? i4_off_sc(r, B) : wb_off_sc(r, WD, B)) + 2 * tok) = sh;
      for (int l = 0; l < r; ++l) {
        float c = 0.f;
        if (l < r_eff) {
          const int col = order[l];
          c = W[col * WS + tok] * rsqrtf(nr[col]) * sqrtf(sqrtf(nr[col]) * unscale);
          if ((sign_bits >> l) & 1u) c = -c;
        }
        gout[(FMT == LOCKS_FMT_I4 ? i4_off_coef(r) : wb_off_coef(r, WD)) + tok * r + l] = (uint8_t)((int)round_code(c, sc, 127.f) + 128);
      }
    }
  }
  // centroid
  if (FMT == LOCKS_FMT_F32) {
    *reinterpret_cast<float4 *>(fout + lane * 4) = make_float4(mu[0], mu[1], mu[2], mu[3]);
  } else {
    float mx = fmaxf(fmaxf(fabsf(mu[0]), fabsf(mu[1])), fmaxf(fabsf(mu[2]), fabsf(mu[3])));
    mx = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
    const __half sh = __float2half_rn(mx / 127.f);
    const float sc = inv_scale(__half2float(sh));
    const int osmu = FMT == LOCKS_FMT_I4 ? i4_off_smu(r, B) : wb_off_smu(r, WD, B);
    if (lane == 0) *reinterpret_cast<__half *>(gout + osmu) = sh;
    uint32_t by[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) by[c] = (uint32_t)((int)round_code(mu[c], sc, 127.f) + 128);
    if (FMT == LOCKS_FMT_I4)   // dim offset c = 2*half + e -> byte e*2 + half, as at B = 16
      *reinterpret_cast<uint32_t *>(gout + i4_off_mu(r, B) + lane * 4) = by[0] | (by[2] << 8) | (by[1] << 16) | (by[3] << 24);
    else
      *reinterpret_cast<uint32_t *>(gout + wb_off_mu(r, WD, B) + lane * 4) = by[0] | (by[1] << 8) | (by[2] << 16) | (by[3] << 24);
    for (int e = osmu + 2 + lane; e < p.S; e += 32) gout[e] = 0;
  }
}

}  // namespace

int locks_launch_build(locks_ctx *c, const locks_kv *kv, int batch, const int32_t *pb, const int32_t *pe,
                       int just_filled, void *summaries, const void *k_new, const int32_t *append_pos,
                       cudaStream_t st, const void *const *k_layers, void *const *summ_layers, int num_layers) {
  BuildParams p;
  p.k = kv->k; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.page_begin = pb; p.page_end = pe;
  p.summ = reinterpret_cast<uint8_t *>(summaries); p.status = c->status;
  p.batch = batch; p.Hkv = c->cfg.num_kv_heads; p.Pmax = c->Pmax; p.num_blocks = kv->num_blocks;
  p.r = c->cfg.rank; p.S = c->S; p.just_filled = just_filled;
  p.k_layers = just_filled ? nullptr : k_layers; p.summ_layers = just_filled ? nullptr : summ_layers;
  p.k_new = just_filled ? k_new : nullptr; p.append_pos = just_filled ? append_pos : nullptr;
  p.hint = nullptr; p.kpages = c->k; p.hint_wpp = 1; p.hint_rounds = 1; p.hint_W = 1;
  if (just_filled && c->hint_dev && c->cfg.summary_fmt == LOCKS_FMT_I4 && c->cfg.q_dtype == LOCKS_BF16) {
    const locks_scan_geom geo = locks_scan_geometry(c, batch);
    p.hint = c->hint_dev; p.hint_wpp = geo.wpp; p.hint_rounds = geo.rounds; p.hint_W = geo.W;
  }
  if (c->B != LOCKS_B) {   // pages of 32 / 64 tokens: the plain kernel (row-major formats; one layer per launch)
    if (k_layers) return LOCKS_ERR_UNSUPPORTED;
    const int B = c->B, smem = build_wide_smem(B);
    const dim3 grid = just_filled ? dim3(batch * p.Hkv) : dim3(c->Pmax, p.Hkv, batch);
    const bool bf16kv = c->cfg.kv_dtype == LOCKS_BF16;
#define LOCKS_WIDE_CASE(F_)                                                                                              \
  do {                                                                                                                  \
    if (locks_attrs_needed(LOCKS_ATTR_BUILD_WIDE + F_)) {                                                                \
      cudaFuncSetAttribute(build_wide_kernel<__nv_bfloat16, F_>, cudaFuncAttributeMaxDynamicSharedMemorySize, build_wide_smem(64)); \
      cudaFuncSetAttribute(build_wide_kernel<float, F_>, cudaFuncAttributeMaxDynamicSharedMemorySize, build_wide_smem(64));         \
    }                                                                                                                   \
    if (bf16kv) build_wide_kernel<__nv_bfloat16, F_><<<grid, 32, smem, st>>>(p, B, just_filled);                        \
    else build_wide_kernel<float, F_><<<grid, 32, smem, st>>>(p, B, just_filled);                                       \
  } while (0)
    switch (c->cfg.summary_fmt) {
      case LOCKS_FMT_I4: LOCKS_WIDE_CASE(LOCKS_FMT_I4); break;
      case LOCKS_FMT_I8: LOCKS_WIDE_CASE(LOCKS_FMT_I8); break;
      case LOCKS_FMT_BF16: LOCKS_WIDE_CASE(LOCKS_FMT_BF16); break;
      default: LOCKS_WIDE_CASE(LOCKS_FMT_F32); break;
    }
#undef LOCKS_WIDE_CASE
    return locks_check_launch(c);
  }
  constexpr int kPer = kBuildWarps * kBuildItems;   // items per CTA (bulk)
  dim3 grid = just_filled ? dim3((batch * p.Hkv + kBuildWarps - 1) / kBuildWarps)
                          : dim3((c->Pmax + kPer - 1) / kPer, p.Hkv, batch * (k_layers ? num_layers : 1));
  const bool bf = c->cfg.kv_dtype == LOCKS_BF16;
  const int smem = kBuildWarps * kBuildSmemPerWarp;
#define LOCKS_BUILD_CASE(F_)                                                                                                \
  do {                                                                                                                     \
    if (bf && just_filled) build_kernel<__nv_bfloat16, F_, true><<<grid, kBuildWarps * 32, smem, st>>>(p);                \
    else if (bf) build_kernel<__nv_bfloat16, F_, false><<<grid, kBuildWarps * 32, smem, st>>>(p);                          \
    else if (just_filled) build_kernel<float, F_, true><<<grid, kBuildWarps * 32, smem, st>>>(p);                          \
    else build_kernel<float, F_, false><<<grid, kBuildWarps * 32, smem, st>>>(p);                                          \
  } while (0)
  switch (c->cfg.summary_fmt) {
    case LOCKS_FMT_I4: LOCKS_BUILD_CASE(LOCKS_FMT_I4); break;
    case LOCKS_FMT_I8: LOCKS_BUILD_CASE(LOCKS_FMT_I8); break;
    case LOCKS_FMT_BF16: LOCKS_BUILD_CASE(LOCKS_FMT_BF16); break;
    default: LOCKS_BUILD_CASE(LOCKS_FMT_F32); break;
  }
#undef LOCKS_BUILD_CASE
  return locks_check_launch(c);
}
