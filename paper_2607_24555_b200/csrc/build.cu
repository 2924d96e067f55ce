// Summary build (Sec. 4 "Build (once, when a page completes)").
//
// build_kernel: one warp per (page, KV head).
//   1. load the page's 16 keys (lane owns 4 consecutive dims of every key), centroid mu, deviations D
//   2. Gram M = D D^T (16 x 16) from shared memory
//   3. eigendecomposition of M by parallel-ordered cyclic Jacobi in fp32 (8 disjoint rotations per
//      round, 15 rounds per sweep, round-robin pairing), eigenvectors accumulated in U; both matrices
//      live in registers, one shared-memory exchange per round
//   4. rank by eigenvalue, keep r_eff <= min(r, 15) modes above the zero-mode thresholds
//   5. V = D^T U_r Sigma_r^-1 (lane's 4 dims), C = U_r Sigma_r, sign: largest |V| entry positive
//   6. store fp32 (F32 format) or quantise: symmetric abs-max, fp16 scale, round-half-even codes
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
};

constexpr int kBuildWarps = 4;
constexpr int kDStride = LOCKS_D + 4;                            // padded row of D in shared memory
constexpr int kBuildSmemPerWarp = (LOCKS_B * kDStride + 2 * LOCKS_B * 17 + 64) * 4 + i4_stride(8);

__device__ __forceinline__ float round_code(float x, float scale, float qmax) {
  if (scale == 0.f) return 0.f;
  float c = rintf(__fdiv_rn(x, scale));
  return fminf(fmaxf(c, -qmax), qmax);
}

template <typename T, int FMT>
__global__ void __launch_bounds__(kBuildWarps * 32) build_kernel(BuildParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int b, h, page;
  bool last_from_new = false;   // row 15 of the page is this step's token
  if (p.just_filled && p.hint && blockIdx.x == 0 && warp == 0)
    locks_update_partition_hint(p.hint, p.seq_lens, p.batch, p.Hkv, p.kpages, p.hint_wpp, p.hint_rounds, p.hint_W, lane);
  if (p.just_filled) {
    const int prob = blockIdx.x * kBuildWarps + warp;
    if (prob >= p.batch * p.Hkv) return;
    b = prob / p.Hkv; h = prob - b * p.Hkv;
    const int Tb = p.seq_lens[b];
    if (Tb <= 0 || (Tb % LOCKS_B) != 0) return;
    page = Tb / LOCKS_B - 1;
    last_from_new = p.k_new && p.append_pos && p.append_pos[b] == Tb - 1;
  } else {
    b = blockIdx.z; h = blockIdx.y;
    const int complete = p.seq_lens[b] / LOCKS_B;
    const int p0 = p.page_begin ? p.page_begin[b] : 0;
    const int p1 = min(p.page_end ? p.page_end[b] : complete, complete);
    page = p0 + blockIdx.x * kBuildWarps + warp;
    if (page < 0 || page >= p1) return;
  }
  if (page >= p.Pmax) return;
  const int block = p.block_table[(int64_t)b * p.Pmax + page];
  if (block < 0 || block >= p.num_blocks) {
    if (lane == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
    return;
  }
  float *Ds = reinterpret_cast<float *>(smem_raw + warp * kBuildSmemPerWarp);   // [16][kDStride]
  float *A = Ds + LOCKS_B * kDStride;                                             // [16][17]
  float *U = A + LOCKS_B * 17;                                                    // [16][17]
  float *rot = U + LOCKS_B * 17;                                                  // c[8], s[8], misc
  uint8_t *blob = reinterpret_cast<uint8_t *>(rot + 64);
  const int r = p.r;

  // ---- 1. load, centre
  const T *K = reinterpret_cast<const T *>(p.k) + (int64_t)block * p.sb + (int64_t)h * p.sh;
  const T *Knew = reinterpret_cast<const T *>(p.k_new) + ((int64_t)b * p.Hkv + h) * LOCKS_D;
  float kv[LOCKS_B][4], mu[4] = {0.f, 0.f, 0.f, 0.f};
  float knorm2 = 0.f;
#pragma unroll
  for (int i = 0; i < LOCKS_B; ++i) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      kv[i][u] = (i == LOCKS_B - 1 && last_from_new) ? ldf<T>(Knew, lane * 4 + u) : ldf<T>(K, (int64_t)i * p.st + lane * 4 + u);
      mu[u] += kv[i][u];
      knorm2 += kv[i][u] * kv[i][u];
    }
  }
  knorm2 = warp_sum(knorm2);
#pragma unroll
  for (int u = 0; u < 4; ++u) mu[u] *= (1.f / LOCKS_B);
#pragma unroll
  for (int i = 0; i < LOCKS_B; ++i) {
#pragma unroll
    for (int u = 0; u < 4; ++u) kv[i][u] -= mu[u];
    *reinterpret_cast<float4 *>(Ds + i * kDStride + lane * 4) = make_float4(kv[i][0], kv[i][1], kv[i][2], kv[i][3]);
  }
  __syncwarp();
  // ---- 2. Gram: lane computes entries e = lane + 32 m -> (i = e / 16, j = e % 16)
#pragma unroll 1
  for (int m = 0; m < 8; ++m) {
    const int e = lane + 32 * m, i = e >> 4, j = e & 15;
    const float4 *ri = reinterpret_cast<const float4 *>(Ds + i * kDStride);
    const float4 *rj = reinterpret_cast<const float4 *>(Ds + j * kDStride);
    float s = 0.f;
    for (int c = 0; c < LOCKS_D / 4; ++c) {
      const float4 a = ri[c], bb = rj[c];
      s += a.x * bb.x + a.y * bb.y + a.z * bb.z + a.w * bb.w;
    }
    A[i * 17 + j] = s;
    U[i * 17 + j] = (i == j) ? 1.f : 0.f;
  }
  __syncwarp();
  // ---- 3. parallel cyclic Jacobi, matrix held in registers.
  // "Slot" space: the 8 rotations of a round always act on the slot pairs (2m, 2m+1); between rounds the 16
  // indices move through the slots by the fixed round-robin permutation `next_slot` (slot 0 stays, the others
  // go round the circle), so that 15 rounds pair every two indices once.  Lane (m = lane / 4, k = lane % 4) holds
  // rows 2m, 2m+1 x columns 4k .. 4k+3 of A (two 2x2 blocks) and of U (rows = tokens, columns = slots).  A round
  // is: rotation angles at the lanes that hold a diagonal block, six shuffles to hand them to the rows and
  // columns they act on, the block updates in registers, and one pass through shared memory (ping-pong
  // buffers, one warp barrier) that applies the permutation.
  {
    const int m = lane >> 2, k = lane & 3;
    auto next_slot = [](int x) { return x == 0 ? 0 : (x == 1 ? 2 : (x == 14 ? 15 : ((x & 1) ? x - 2 : x + 2))); };
    constexpr int kJS = 20;   // row stride of the exchange buffers (16-byte aligned rows)
    float *buf0 = Ds, *buf1 = Ds + 2 * LOCKS_B * kJS;   // each: A[16][kJS] then U[16][kJS]
    float a[8], u[8];   // index = 4 * blk + 2 * rowbit + colbit, columns 4k + 2 blk + colbit
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int i = 2 * m + ((e >> 1) & 1), j = 4 * k + 2 * (e >> 2) + (e & 1);
      a[e] = A[i * 17 + j];
      u[e] = (i == j) ? 1.f : 0.f;
    }
    int wr_row[2], wr_col[4];   // where this lane's rows / columns go after a round
#pragma unroll
    for (int rb = 0; rb < 2; ++rb) wr_row[rb] = next_slot(2 * m + rb);
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) wr_col[c4] = next_slot(4 * k + c4);
    const bool diag_lane = k == (m >> 1);
    const int dblk = m & 1;             // which of the two blocks is the diagonal one (diag lanes)
    const int src_row = m * 4 + (m >> 1);           // lane holding the diagonal block of row pair m
    const int src_c0 = 9 * k, src_c1 = 9 * k + 4;   // ... of column pairs 2k and 2k + 1
    // The rotations square matrix entries: bring the matrix to unit scale first (an exact power of two, taken
    // from its largest entry and undone on the eigenvalues), so that keys of any magnitude are handled alike.
    float unscale = 1.f;
    {
      float amax = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(a[e]));
      amax = warp_max(amax);
      if (amax > 0.f && amax < INFINITY) {
        int ex;
        (void)frexpf(amax, &ex);
        ex = max(-120, min(120, ex));
        const float sc = ldexpf(1.f, -ex);
        unscale = ldexpf(1.f, ex);
#pragma unroll
        for (int e = 0; e < 8; ++e) a[e] *= sc;
      }
    }
    float normA = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) normA += a[e] * a[e];
    normA = warp_sum(normA);
    int parity = 0;
    for (int sweep = 0; sweep < 12; ++sweep) {
      float off = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const bool on_diag = diag_lane && (e >> 2) == dblk && (((e >> 1) & 1) == (e & 1));
        off += on_diag ? 0.f : a[e] * a[e];
      }
      off = warp_sum(off);
      if (off <= 1e-13f * normA || normA == 0.f) break;
#pragma unroll 1
      for (int round = 0; round < 15; ++round) {
        // rotation of the slot pair held as a diagonal block (other lanes compute on whatever they hold; unused)
        const float app = dblk ? a[4] : a[0], apq = dblk ? a[5] : a[1], aqq = dblk ? a[7] : a[3];
        float c = 1.f, sn = 0.f;
        {
          // tan of the rotation angle: t = 2 apq / (d + sign(d) sqrt(d^2 + 4 apq^2)), d = aqq - app (the smaller
          // root).  Approximate root and division are enough for the angle; c^2 + s^2 = 1 comes from the last
          // two lines.  Entries too small to square are left alone.
          const float d = aqq - app, h = d * d + 4.f * apq * apq;
          if (h > 1e-37f && h < 1e37f) {
            const float tt = __fdividef(2.f * apq, d + copysignf(h * rsqrtf(h), d));
            c = rsqrtf(tt * tt + 1.f);
            sn = tt * c;
          }
        }
        const float cr = __shfl_sync(0xffffffffu, c, src_row), sr = __shfl_sync(0xffffffffu, sn, src_row);
        const float cc[2] = {__shfl_sync(0xffffffffu, c, src_c0), __shfl_sync(0xffffffffu, c, src_c1)};
        const float sc[2] = {__shfl_sync(0xffffffffu, sn, src_c0), __shfl_sync(0xffffffffu, sn, src_c1)};
        float *dst = parity ? buf1 : buf0;
#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {
          float *x = a + 4 * blk, *y = u + 4 * blk;
          // columns: [x_ip x_iq] <- [c x_ip - s x_iq, s x_ip + c x_iq]
          const float t00 = cc[blk] * x[0] - sc[blk] * x[1], t01 = sc[blk] * x[0] + cc[blk] * x[1];
          const float t10 = cc[blk] * x[2] - sc[blk] * x[3], t11 = sc[blk] * x[2] + cc[blk] * x[3];
          // rows: [x_pj; x_qj] <- [c x_pj - s x_qj; s x_pj + c x_qj]
          x[0] = cr * t00 - sr * t10; x[1] = cr * t01 - sr * t11;
          x[2] = sr * t00 + cr * t10; x[3] = sr * t01 + cr * t11;
          const float v00 = cc[blk] * y[0] - sc[blk] * y[1], v01 = sc[blk] * y[0] + cc[blk] * y[1];
          const float v10 = cc[blk] * y[2] - sc[blk] * y[3], v11 = sc[blk] * y[2] + cc[blk] * y[3];
          y[0] = v00; y[1] = v01; y[2] = v10; y[3] = v11;
        }
        // the permutation: A rows and columns, U columns
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int rb = (e >> 1) & 1, c4 = 2 * (e >> 2) + (e & 1);
          dst[wr_row[rb] * kJS + wr_col[c4]] = a[e];
          dst[LOCKS_B * kJS + (2 * m + rb) * kJS + wr_col[c4]] = u[e];
        }
        __syncwarp();
#pragma unroll
        for (int rb = 0; rb < 2; ++rb) {   // columns 4k .. 4k+3 of a row are one 16-byte read
          const float4 ra = *reinterpret_cast<const float4 *>(dst + (2 * m + rb) * kJS + 4 * k);
          const float4 ru = *reinterpret_cast<const float4 *>(dst + LOCKS_B * kJS + (2 * m + rb) * kJS + 4 * k);
          a[2 * rb] = ra.x; a[2 * rb + 1] = ra.y; a[4 + 2 * rb] = ra.z; a[4 + 2 * rb + 1] = ra.w;
          u[2 * rb] = ru.x; u[2 * rb + 1] = ru.y; u[4 + 2 * rb] = ru.z; u[4 + 2 * rb + 1] = ru.w;
        }
        parity ^= 1;
      }
    }
    __syncwarp();
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int i = 2 * m + ((e >> 1) & 1), j = 4 * k + 2 * (e >> 2) + (e & 1);
      A[i * 17 + j] = a[e] * unscale;
      U[i * 17 + j] = u[e];
    }
    __syncwarp();
  }
  // ---- 4. order the eigenvalues (descending, ties by index), choose r_eff
  float lam = (lane < 16) ? A[lane * 17 + lane] : -INFINITY;
  int rank = 0;
  for (int j = 0; j < 16; ++j) {
    const float lj = __shfl_sync(0xffffffffu, lam, j);
    rank += (lj > lam) || (lj == lam && j < lane);
  }
  if (lane < 16) { reinterpret_cast<int *>(rot)[32 + rank] = lane; rot[48 + rank] = lam; }
  __syncwarp();
  const float lam0 = rot[48];
  int r_eff = 0;
  const int rmax = min(r, LOCKS_B - 1);
  for (int l = 0; l < rmax; ++l) {
    const float ll = rot[48 + l];
    if (lam0 > 0.f && ll > 1e-6f * lam0 && ll > 1e-10f * knorm2) r_eff = l + 1; else break;
  }
  // ---- 5/6. per mode: basis entries of this lane's 4 dims, sign, quantise
  if (FMT == LOCKS_FMT_I4) {
    for (int e = lane; e < i4_stride(8) / 4; e += 32) reinterpret_cast<uint32_t *>(blob)[e] = 0u;
    __syncwarp();
  }
  float *fout = reinterpret_cast<float *>(p.summ + ((int64_t)block * p.Hkv + h) * p.S);
  float csign[16];
#pragma unroll 1
  for (int l = 0; l < r; ++l) {
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    float sgn = 1.f;
    if (l < r_eff) {
      const int col = reinterpret_cast<int *>(rot)[32 + l];
      const float inv = rsqrtf(rot[48 + l]);
#pragma unroll
      for (int i = 0; i < LOCKS_B; ++i) {
        const float u = U[i * 17 + col];
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] += kv[i][c] * u;
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] *= inv;
      // sign: entry of largest magnitude (lowest dim on ties) positive
      float best = fabsf(v[0]); int bi = lane * 4; float bv = v[0];
#pragma unroll
      for (int c = 1; c < 4; ++c) if (fabsf(v[c]) > best) { best = fabsf(v[c]); bi = lane * 4 + c; bv = v[c]; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; bv = ov; }
      }
      if (bv < 0.f) sgn = -1.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] *= sgn;
    }
    csign[l & 15] = sgn;
    if (FMT == LOCKS_FMT_F32) {
      *reinterpret_cast<float4 *>(fout + LOCKS_D + l * LOCKS_D + lane * 4) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
      float mx = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
      mx = warp_max(mx);
      const __half sh = __float2half_rn(mx / 7.f);
      const float sc = __half2float(sh);
      if (lane == 0) *reinterpret_cast<__half *>(blob + i4_off_sv(r) + 2 * l) = sh;
      // lane = 8 t + s owns dims 32 t + 4 s + {0,1,2,3} = (half, e) in {0,1}^2 of k-step s
      const int t = lane >> 3, s = lane & 7, i0 = (s & 1) << 1;
      uint32_t n[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) n[c] = (uint32_t)((int)round_code(v[c], sc, 7.f) + 8);
      // dim offset c = 2*half + e -> nibble i0 + half + 4 e
      uint32_t pw = (n[0] << (4 * i0)) | (n[1] << (4 * (i0 + 4))) | (n[2] << (4 * (i0 + 1))) | (n[3] << (4 * (i0 + 5)));
      pw |= __shfl_xor_sync(0xffffffffu, pw, 1);
      if ((s & 1) == 0) *reinterpret_cast<uint32_t *>(blob + (l * 4 + t) * 16 + (s >> 1) * 4) = pw;
    }
  }
  // coefficients: lane i < 16 owns token i
  if (lane < LOCKS_B) {
    float cf[16];
    float mx = 0.f;
    for (int l = 0; l < r; ++l) {
      float c = 0.f;
      if (l < r_eff) c = sqrtf(rot[48 + l]) * U[lane * 17 + reinterpret_cast<int *>(rot)[32 + l]] * csign[l & 15];
      cf[l & 15] = c;
      mx = fmaxf(mx, fabsf(c));
    }
    if (FMT == LOCKS_FMT_F32) {
      for (int l = 0; l < r; ++l) fout[LOCKS_D + r * LOCKS_D + lane * r + l] = cf[l & 15];
    } else {
      const __half sh = __float2half_rn(mx / 127.f);
      const float sc = __half2float(sh);
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
  } else {
    float mx = fmaxf(fmaxf(fabsf(mu[0]), fabsf(mu[1])), fmaxf(fabsf(mu[2]), fabsf(mu[3])));
    mx = warp_max(mx);
    const __half sh = __float2half_rn(mx / 127.f);
    const float sc = __half2float(sh);
    if (lane == 0) *reinterpret_cast<__half *>(blob + i4_off_smu(r)) = sh;
    uint32_t bytes[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) bytes[c] = (uint32_t)((int)round_code(mu[c], sc, 127.f) + 128);
    // dim offset c = 2*half + e -> byte e*2 + half
    const uint32_t w = bytes[0] | (bytes[2] << 8) | (bytes[1] << 16) | (bytes[3] << 24);
    *reinterpret_cast<uint32_t *>(blob + i4_off_mu(r) + lane * 4) = w;
    __syncwarp();
    uint4 *dst = reinterpret_cast<uint4 *>(p.summ + ((int64_t)block * p.Hkv + h) * p.S);
    for (int e = lane; e < p.S / 16; e += 32) dst[e] = reinterpret_cast<const uint4 *>(blob)[e];
  }
}

}  // namespace

int locks_launch_build(locks_ctx *c, const locks_kv *kv, int batch, const int32_t *pb, const int32_t *pe,
                       int just_filled, void *summaries, const void *k_new, const int32_t *append_pos,
                       cudaStream_t st) {
  BuildParams p;
  p.k = kv->k; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.page_begin = pb; p.page_end = pe;
  p.summ = reinterpret_cast<uint8_t *>(summaries); p.status = c->status;
  p.batch = batch; p.Hkv = c->cfg.num_kv_heads; p.Pmax = c->Pmax; p.num_blocks = kv->num_blocks;
  p.r = c->cfg.rank; p.S = c->S; p.just_filled = just_filled;
  p.k_new = just_filled ? k_new : nullptr; p.append_pos = just_filled ? append_pos : nullptr;
  p.hint = nullptr; p.kpages = c->k; p.hint_wpp = 1; p.hint_rounds = 1; p.hint_W = 1;
  if (just_filled && c->hint_dev && c->cfg.summary_fmt == LOCKS_FMT_I4 && c->cfg.q_dtype == LOCKS_BF16) {
    const locks_scan_geom geo = locks_scan_geometry(c, batch);
    p.hint = c->hint_dev; p.hint_wpp = geo.wpp; p.hint_rounds = geo.rounds; p.hint_W = geo.W;
  }
  dim3 grid = just_filled ? dim3((batch * p.Hkv + kBuildWarps - 1) / kBuildWarps)
                          : dim3((c->Pmax + kBuildWarps - 1) / kBuildWarps, p.Hkv, batch);
  const int smem = kBuildWarps * kBuildSmemPerWarp;
  const bool bf = c->cfg.kv_dtype == LOCKS_BF16, i4 = c->cfg.summary_fmt == LOCKS_FMT_I4;
  if (locks_attrs_needed(LOCKS_ATTR_BUILD)) {
    cudaFuncSetAttribute(build_kernel<__nv_bfloat16, LOCKS_FMT_I4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaFuncSetAttribute(build_kernel<__nv_bfloat16, LOCKS_FMT_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaFuncSetAttribute(build_kernel<float, LOCKS_FMT_I4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaFuncSetAttribute(build_kernel<float, LOCKS_FMT_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  }
  if (bf && i4) build_kernel<__nv_bfloat16, LOCKS_FMT_I4><<<grid, kBuildWarps * 32, smem, st>>>(p);
  else if (bf) build_kernel<__nv_bfloat16, LOCKS_FMT_F32><<<grid, kBuildWarps * 32, smem, st>>>(p);
  else if (i4) build_kernel<float, LOCKS_FMT_I4><<<grid, kBuildWarps * 32, smem, st>>>(p);
  else build_kernel<float, LOCKS_FMT_F32><<<grid, kBuildWarps * 32, smem, st>>>(p);
  return locks_check_launch(c);
}
