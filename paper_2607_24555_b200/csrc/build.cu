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

#ifndef LOCKS_BUILD_OFF_TOL
#define LOCKS_BUILD_OFF_TOL 1e-13f   // squared off-diagonal norm over squared norm at which the sweeps stop
#endif
#ifndef LOCKS_BUILD_SWEEPS
#define LOCKS_BUILD_SWEEPS 12   // upper bound; a page stops as soon as its off-diagonal norm is at rounding level
#endif
constexpr int kBuildWarps = 3;
constexpr int kBuildCtasPerSm = 6;                               // 18 warps per SM (bf16 keys: 11.3 KB per warp)
constexpr int kBuildScratch = 2 * 2 * LOCKS_B * LOCKS_B * 4;      // 4096 B: bf16 half-tiles of D (hi | lo), then the exchange buffers
template <typename T> __host__ __device__ constexpr int build_smem_per_warp() {      // raw key tile + scratch + A, U + misc + blob
  return LOCKS_B * LOCKS_D * (int)sizeof(T) + kBuildScratch + (2 * LOCKS_B * 17 + 64) * 4 + i4_stride(8);
}
// Placement of a 16 x 16 matrix in an exchange buffer.  A round writes entry (row, column) with rows and
// columns permuted (32 lanes x one scalar store: 8 rows x 4 columns) and reads it back row by row (8 rows x 4
// columns again), 32 instructions per round in all, so bank conflicts are what a round costs.  The placement
// below makes every one of those instructions conflict-free: bank = 4 f(row) + g(column), where f takes each of
// its 8 values on two rows that never meet in one instruction (one even, one odd, on either side of the
// permutation) and g takes each of its 4 values on four columns that never meet either.
__device__ __forceinline__ int jrow_part(int r) {   // 128 (odd row) + 4 f(r)
  const int f = (r & 1) ? (r == 15 ? 1 : (r == 1 ? 0 : (r + 1) >> 1)) : (r >> 1);
  return ((r & 1) << 7) + 4 * f;
}
__device__ __forceinline__ int jcol_part(int c) {   // 32 (c mod 4) + g(c)
  const int g = ((c & 3) == 3) ? (((c + 1) >> 2) & 3) : (c >> 2);
  return ((c & 3) << 5) + g;
}

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

template <typename T, int FMT>
__global__ void __launch_bounds__(kBuildWarps * 32, kBuildCtasPerSm) build_kernel(BuildParams p) {
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
  // Loops over the 16 keys stay rolled: a warp runs through this code once per page, and when a page fills inside
  // a decode step the code is cold, so its length in instructions is part of the latency.  The page's keys are
  // staged in shared memory once and every phase reads them from there.
  constexpr int kRawBytes = LOCKS_B * LOCKS_D * (int)sizeof(T);
  constexpr int kRowBytes = LOCKS_D * (int)sizeof(T);
  uint8_t *raw = smem_raw + warp * build_smem_per_warp<T>();                      // [16][128] keys as stored
  uint8_t *scratch = raw + kRawBytes;                                             // D half-tiles, then exchange buffers
  float *A = reinterpret_cast<float *>(scratch + kBuildScratch);                 // [16][17]
  float *U = A + LOCKS_B * 17;                                                    // [16][17] (first: the cross product)
  float *rot = U + LOCKS_B * 17;                                                  // misc
  uint8_t *blob = reinterpret_cast<uint8_t *>(rot + 64);
  float *mus = reinterpret_cast<float *>(blob);                                   // centroid, until the blob is assembled
  const int r = p.r;

  // ---- 1. stage the keys, centroid
  {
    const uint8_t *K = reinterpret_cast<const uint8_t *>(p.k) + ((int64_t)block * p.sb + (int64_t)h * p.sh) * (int64_t)sizeof(T);
    const uint8_t *Knew = reinterpret_cast<const uint8_t *>(p.k_new) + ((int64_t)b * p.Hkv + h) * kRowBytes;
    constexpr int kCpr = kRowBytes / 16;   // 16-byte chunks per row
#pragma unroll 4
    for (int c = lane; c < LOCKS_B * kCpr; c += 32) {
      const int row = c / kCpr, ch = c - row * kCpr;
      const uint8_t *src = (row == LOCKS_B - 1 && last_from_new) ? Knew : K + (int64_t)row * p.st * (int64_t)sizeof(T);
      cp_async16(raw + c * 16, src + ch * 16, true);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncwarp();
  }
  auto key4 = [&](int row, int d0, float (&v)[4]) {   // keys (row, d0 .. d0 + 3) as fp32
    if (sizeof(T) == 2) {
      const uint2 w = *reinterpret_cast<const uint2 *>(raw + row * kRowBytes + d0 * 2);
      v[0] = __uint_as_float(w.x << 16); v[1] = __uint_as_float(w.x & 0xFFFF0000u);
      v[2] = __uint_as_float(w.y << 16); v[3] = __uint_as_float(w.y & 0xFFFF0000u);
    } else {
      const float4 w = *reinterpret_cast<const float4 *>(raw + row * kRowBytes + d0 * 4);
      v[0] = w.x; v[1] = w.y; v[2] = w.z; v[3] = w.w;
    }
  };
  float mu[4] = {0.f, 0.f, 0.f, 0.f};   // of this lane's dims 4 lane .. 4 lane + 3
  float knorm2 = 0.f;
#pragma unroll 4
  for (int i = 0; i < LOCKS_B; ++i) {
    float v[4];
    key4(i, 4 * lane, v);
#pragma unroll
    for (int u = 0; u < 4; ++u) { mu[u] += v[u]; knorm2 = fmaf(v[u], v[u], knorm2); }
  }
  knorm2 = warp_sum(knorm2);
#pragma unroll
  for (int u = 0; u < 4; ++u) mu[u] *= (1.f / LOCKS_B);
  *reinterpret_cast<float4 *>(mus + 4 * lane) = make_float4(mu[0], mu[1], mu[2], mu[3]);
  __syncwarp();
  // ---- 2. Gram matrix M = D D^T on the tensor cores.  D = H + L with H = bf16(D), L = bf16(D - H) (16 significant
  // bits; the bf16 products are exact and accumulate in fp32): M = (H H^T + L L^T) + H L^T + (H L^T)^T.  The A
  // operand (tokens x dims) and the B operand (dims x tokens) of an m16n8k16 step are the same registers.
  // Two passes over 64 dims each: the half-tiles of H and L (16 rows x 128 bytes, 16-byte chunks XOR-swizzled with
  // the row so that ldmatrix reads are conflict-free) share the 4 KB of scratch.
  {
    float X0[4] = {0.f, 0.f, 0.f, 0.f}, X1[4] = {0.f, 0.f, 0.f, 0.f}, Y0[4] = {0.f, 0.f, 0.f, 0.f}, Y1[4] = {0.f, 0.f, 0.f, 0.f};
    const int rh = lane >> 4, c16 = lane & 15;                      // writer: rows 8 rh .. 8 rh + 7, dims 4 c16 .. + 3 of the half
    const int mq = lane >> 3, rr = lane & 7, tok = (mq & 1) * 8 + rr;   // reader (ldmatrix address lanes)
#pragma unroll 1
    for (int hf = 0; hf < 2; ++hf) {
      const float4 m4 = *reinterpret_cast<const float4 *>(mus + 64 * hf + 4 * c16);
#pragma unroll 2
      for (int i = 0; i < 8; ++i) {
        const int row = 8 * rh + i;
        float v[4];
        key4(row, 64 * hf + 4 * c16, v);
        v[0] -= m4.x; v[1] -= m4.y; v[2] -= m4.z; v[3] -= m4.w;
        const uint32_t h01 = pack_bf16(v[0], v[1]), h23 = pack_bf16(v[2], v[3]);
        const uint32_t l01 = pack_bf16(v[0] - __uint_as_float(h01 << 16), v[1] - __uint_as_float(h01 & 0xFFFF0000u));
        const uint32_t l23 = pack_bf16(v[2] - __uint_as_float(h23 << 16), v[3] - __uint_as_float(h23 & 0xFFFF0000u));
        uint8_t *dst = scratch + row * 128 + ((((c16 >> 1) ^ (row & 7)) << 4) | ((c16 & 1) << 3));
        *reinterpret_cast<uint2 *>(dst) = make_uint2(h01, h23);
        *reinterpret_cast<uint2 *>(dst + 2048) = make_uint2(l01, l23);
      }
      __syncwarp();
#pragma unroll 1
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
    // accumulator (x = lane / 4, t = lane % 4): [0..1] = row x, columns 2t, 2t+1; [2..3] = row x + 8
    const int x = lane >> 2, t = lane & 3;
    A[x * 17 + 2 * t] = X0[0]; A[x * 17 + 2 * t + 1] = X0[1]; A[(x + 8) * 17 + 2 * t] = X0[2]; A[(x + 8) * 17 + 2 * t + 1] = X0[3];
    A[x * 17 + 8 + 2 * t] = X1[0]; A[x * 17 + 9 + 2 * t] = X1[1]; A[(x + 8) * 17 + 8 + 2 * t] = X1[2]; A[(x + 8) * 17 + 9 + 2 * t] = X1[3];
    U[x * 17 + 2 * t] = Y0[0]; U[x * 17 + 2 * t + 1] = Y0[1]; U[(x + 8) * 17 + 2 * t] = Y0[2]; U[(x + 8) * 17 + 2 * t + 1] = Y0[3];
    U[x * 17 + 8 + 2 * t] = Y1[0]; U[x * 17 + 9 + 2 * t] = Y1[1]; U[(x + 8) * 17 + 8 + 2 * t] = Y1[2]; U[(x + 8) * 17 + 9 + 2 * t] = Y1[3];
    __syncwarp();
  }
  // ---- 3. parallel cyclic Jacobi, matrix held in registers.
  // "Slot" space: the 8 rotations of a round always act on the slot pairs (2m, 2m+1); between rounds the 16
  // indices move through the slots by the fixed round-robin permutation `next_slot` (slot 0 stays, the others
  // go round the circle), so that 15 rounds pair every two indices once.  Lane (m = lane / 4, k = lane % 4) holds
  // rows 2m, 2m+1 x columns 4k .. 4k+3 of A (two 2x2 blocks) and of U (rows = tokens, columns = slots).  A round
  // is: rotation angles at the lanes that hold a diagonal block, six shuffles to hand them to the rows and
  // columns they act on, the block updates in registers, and one pass through shared memory (ping-pong
  // buffers, one warp barrier) that applies the permutation.  The two blocks of a lane are updated together:
  // entry (row bit, column bit) of both blocks forms one packed fp32 pair (.x = columns 4k, 4k+1, .y = columns
  // 4k+2, 4k+3), the column rotation multiplies by per-block coefficient pairs, the row rotation by the same
  // coefficient in both halves.
  {
    const int m = lane >> 2, k = lane & 3;
    auto next_slot = [](int x) { return x == 0 ? 0 : (x == 1 ? 2 : (x == 14 ? 15 : ((x & 1) ? x - 2 : x + 2))); };
    float *buf0 = reinterpret_cast<float *>(scratch), *buf1 = buf0 + 2 * LOCKS_B * LOCKS_B;   // each: A then U, 256 floats
    float2 pa[2][2], pu[2][2];   // [row bit][column bit]
#pragma unroll
    for (int rb = 0; rb < 2; ++rb)
#pragma unroll
      for (int cb = 0; cb < 2; ++cb) {
        const int i = 2 * m + rb, j0 = 4 * k + cb, j1 = j0 + 2;
        pa[rb][cb].x = 0.5f * (A[i * 17 + j0] + A[j0 * 17 + i]) + U[i * 17 + j0] + U[j0 * 17 + i];
        pa[rb][cb].y = 0.5f * (A[i * 17 + j1] + A[j1 * 17 + i]) + U[i * 17 + j1] + U[j1 * 17 + i];
        pu[rb][cb].x = (i == j0) ? 1.f : 0.f;
        pu[rb][cb].y = (i == j1) ? 1.f : 0.f;
      }
    __syncwarp();
    // buffer offsets of this lane's entries: where its rows / columns go after a round, and where they are read
    int wr_row[2], wr_col[4], rd_row[2], rd_col[4];
#pragma unroll
    for (int rb = 0; rb < 2; ++rb) { wr_row[rb] = jrow_part(next_slot(2 * m + rb)); rd_row[rb] = jrow_part(2 * m + rb); }
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) { wr_col[c4] = jcol_part(next_slot(4 * k + c4)); rd_col[c4] = jcol_part(4 * k + c4); }
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
      for (int rb = 0; rb < 2; ++rb)
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) amax = fmaxf(amax, fmaxf(fabsf(pa[rb][cb].x), fabsf(pa[rb][cb].y)));
      amax = warp_max(amax);
      if (amax > 0.f && amax < INFINITY) {
        int ex;
        (void)frexpf(amax, &ex);
        ex = max(-120, min(120, ex));
        const float sc = ldexpf(1.f, -ex);
        unscale = ldexpf(1.f, ex);
#pragma unroll
        for (int rb = 0; rb < 2; ++rb)
#pragma unroll
          for (int cb = 0; cb < 2; ++cb) { pa[rb][cb].x *= sc; pa[rb][cb].y *= sc; }
      }
    }
    float normA = 0.f;
#pragma unroll
    for (int rb = 0; rb < 2; ++rb)
#pragma unroll
      for (int cb = 0; cb < 2; ++cb) normA += pa[rb][cb].x * pa[rb][cb].x + pa[rb][cb].y * pa[rb][cb].y;
    normA = warp_sum(normA);
    int parity = 0;
    for (int sweep = 0; sweep < LOCKS_BUILD_SWEEPS; ++sweep) {
      float off = 0.f;
#pragma unroll
      for (int rb = 0; rb < 2; ++rb)
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
          const bool dg = diag_lane && rb == cb;   // diagonal entries of the diagonal block do not count
          off += (dg && dblk == 0) ? 0.f : pa[rb][cb].x * pa[rb][cb].x;
          off += (dg && dblk == 1) ? 0.f : pa[rb][cb].y * pa[rb][cb].y;
        }
      off = warp_sum(off);
      if (off <= LOCKS_BUILD_OFF_TOL * normA || normA == 0.f) break;
#pragma unroll 1
      for (int round = 0; round < 15; ++round) {
        // rotation of the slot pair held as a diagonal block (other lanes compute on whatever they hold; unused)
        const float app = dblk ? pa[0][0].y : pa[0][0].x, apq = dblk ? pa[0][1].y : pa[0][1].x;
        const float aqq = dblk ? pa[1][1].y : pa[1][1].x;
        float c = 1.f, sn = 0.f;
        {
          // The rotation that annihilates apq, smaller angle: with d = aqq - app and h = d^2 + 4 apq^2,
          // cos 2t = |d| / sqrt(h) and sin 2t = 2 apq sign(d) / sqrt(h), so c = sqrt((1 + cos 2t) / 2) and
          // s = sin 2t / (2 c): two reciprocal square roots in a row (approximate ones are enough for the angle;
          // c^2 + s^2 = 1 holds to their rounding).  Entries too small to square are left alone.
          const float d = aqq - app, hh = d * d + 4.f * apq * apq;
          if (hh > 1e-37f && hh < 1e37f) {
            const float rs = rsqrtf(hh);
            const float x = fmaf(0.5f * fabsf(d), rs, 0.5f);
            const float r2 = rsqrtf(x);
            c = x * r2;
            sn = copysignf(apq * rs * r2, apq * d);
            if (d == 0.f) sn = copysignf(fabsf(sn), apq);
          }
        }
        const float cr = __shfl_sync(0xffffffffu, c, src_row), sr = __shfl_sync(0xffffffffu, sn, src_row);
        const float2 Cc = make_float2(__shfl_sync(0xffffffffu, c, src_c0), __shfl_sync(0xffffffffu, c, src_c1));
        const float2 Sc = make_float2(__shfl_sync(0xffffffffu, sn, src_c0), __shfl_sync(0xffffffffu, sn, src_c1));
        const float2 nSc = make_float2(-Sc.x, -Sc.y), Cr = make_float2(cr, cr), Sr = make_float2(sr, sr), nSr = make_float2(-sr, -sr);
        float *dst = parity ? buf1 : buf0;
        // columns: [x_ip x_iq] <- [c x_ip - s x_iq, s x_ip + c x_iq]; rows: [x_pj; x_qj] <- [c x_pj - s x_qj; s x_pj + c x_qj]
        float2 ta[2][2];
#pragma unroll
        for (int rb = 0; rb < 2; ++rb) {
          ta[rb][0] = fma2(Cc, pa[rb][0], mul2(nSc, pa[rb][1]));
          ta[rb][1] = fma2(Sc, pa[rb][0], mul2(Cc, pa[rb][1]));
          const float2 u0 = fma2(Cc, pu[rb][0], mul2(nSc, pu[rb][1]));
          const float2 u1 = fma2(Sc, pu[rb][0], mul2(Cc, pu[rb][1]));
          pu[rb][0] = u0; pu[rb][1] = u1;
        }
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
          pa[0][cb] = fma2(Cr, ta[0][cb], mul2(nSr, ta[1][cb]));
          pa[1][cb] = fma2(Sr, ta[0][cb], mul2(Cr, ta[1][cb]));
        }
        // the permutation: A rows and columns, U columns
#pragma unroll
        for (int rb = 0; rb < 2; ++rb)
#pragma unroll
          for (int cb = 0; cb < 2; ++cb) {
            dst[wr_row[rb] + wr_col[cb]] = pa[rb][cb].x;
            dst[wr_row[rb] + wr_col[2 + cb]] = pa[rb][cb].y;
            dst[LOCKS_B * LOCKS_B + rd_row[rb] + wr_col[cb]] = pu[rb][cb].x;
            dst[LOCKS_B * LOCKS_B + rd_row[rb] + wr_col[2 + cb]] = pu[rb][cb].y;
          }
        __syncwarp();
#pragma unroll
        for (int rb = 0; rb < 2; ++rb)
#pragma unroll
          for (int cb = 0; cb < 2; ++cb) {
            pa[rb][cb] = make_float2(dst[rd_row[rb] + rd_col[cb]], dst[rd_row[rb] + rd_col[2 + cb]]);
            pu[rb][cb] = make_float2(dst[LOCKS_B * LOCKS_B + rd_row[rb] + rd_col[cb]], dst[LOCKS_B * LOCKS_B + rd_row[rb] + rd_col[2 + cb]]);
          }
        parity ^= 1;
      }
    }
    __syncwarp();
#pragma unroll
    for (int rb = 0; rb < 2; ++rb)
#pragma unroll
      for (int cb = 0; cb < 2; ++cb) {
        const int i = 2 * m + rb, j0 = 4 * k + cb, j1 = j0 + 2;
        A[i * 17 + j0] = pa[rb][cb].x * unscale; A[i * 17 + j1] = pa[rb][cb].y * unscale;
        U[i * 17 + j0] = pu[rb][cb].x; U[i * 17 + j1] = pu[rb][cb].y;
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
  uint8_t *gout = p.summ + ((int64_t)block * p.Hkv + h) * p.S;
  float *fout = reinterpret_cast<float *>(gout);
  uint32_t sign_bits = 0u;   // bit l: mode l was flipped
  {
#pragma unroll 1
    for (int l = 0; l < r; ++l) {
      float v[4] = {0.f, 0.f, 0.f, 0.f};
      float best = 0.f;   // largest magnitude of the mode's basis vector
      if (l < r_eff) {
        const int col = reinterpret_cast<int *>(rot)[32 + l];
        const float inv = rsqrtf(rot[48 + l]);
#pragma unroll
        for (int i = 0; i < LOCKS_B; ++i) {
          const float u = U[i * 17 + col];
          float kd[4];
          key4(i, 4 * lane, kd);
#pragma unroll
          for (int c = 0; c < 4; ++c) v[c] = fmaf(kd[c] - mu[c], u, v[c]);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] *= inv;
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
        uint32_t w = 0u;
#pragma unroll
        for (int c = 0; c < 4; ++c) w |= (uint32_t)((int)round_code(v[c], sc, 127.f) + 128) << (8 * c);
        *reinterpret_cast<uint32_t *>(gout + l * LOCKS_D + lane * 4) = w;
      } else {
        const __half sh = __float2half_rn(best / 7.f);
        const float sc = inv_scale(__half2float(sh));
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
  }
  // coefficients: lane i < 16 owns token i
  if (lane < LOCKS_B) {
    float cf[16];
    float mx = 0.f;
    for (int l = 0; l < r; ++l) {
      float c = 0.f;
      if (l < r_eff) {
        c = sqrtf(rot[48 + l]) * U[lane * 17 + reinterpret_cast<int *>(rot)[32 + l]];
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
    uint32_t w = 0u;
#pragma unroll
    for (int c = 0; c < 4; ++c) w |= (uint32_t)((int)round_code(mu[c], sc, 127.f) + 128) << (8 * c);
    *reinterpret_cast<uint32_t *>(gout + wb_off_mu(r, W) + lane * 4) = w;
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
  const bool bf = c->cfg.kv_dtype == LOCKS_BF16;
  const int smem_bf = kBuildWarps * build_smem_per_warp<__nv_bfloat16>(), smem_f32 = kBuildWarps * build_smem_per_warp<float>();
  const int smem = bf ? smem_bf : smem_f32;
#define LOCKS_BUILD_CASE(F_)                                                                                                \
  do {                                                                                                                     \
    if (locks_attrs_needed(LOCKS_ATTR_BUILD + F_)) {                                                                       \
      cudaFuncSetAttribute(build_kernel<__nv_bfloat16, F_>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bf);       \
      cudaFuncSetAttribute(build_kernel<float, F_>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_f32);               \
    }                                                                                                                      \
    if (bf) build_kernel<__nv_bfloat16, F_><<<grid, kBuildWarps * 32, smem, st>>>(p);                                     \
    else build_kernel<float, F_><<<grid, kBuildWarps * 32, smem, st>>>(p);                                                 \
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
