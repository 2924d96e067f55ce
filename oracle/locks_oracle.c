/*
 * LOCKS oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the page-local spectral-summary selector computes,
 * written from the paper's definitions.  It shares no code, header, table or helper with the
 * CUDA library; only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Paper passages followed (section / equation names of the LOCKS paper):
 *   - "Build (once, when a page completes)" in Sec. 4: centre the page, eigendecompose the
 *     B x B Gram of the deviations, keep r modes: C = U_r Sigma_r, V = D^T U_r Sigma_r^{-1};
 *     zero modes dropped, their coefficients zero; int4 basis, int8 coefficients and centroid,
 *     per-column / per-row scales.
 *   - Eq. (1): s^_j(q) = log sum_{i in P_j} exp[(q.mu_j + (V_j^T q).c_i)/sqrt(d)].
 *   - share-average combine (Sec. 4): m^_g(j) = exp(s^_j(q_g)) / sum_j' exp(s^_j'(q_g)),
 *     m_bar_j = (1/G) sum_g m^_g(j); sink + most recent page fill two of k = ceil(b/B) slots,
 *     top-(k-2) of the remaining pages by m_bar_j fill the rest.
 *   - Sec. 3 "Decode-time attention": o = sum_i softmax_i(q.k_i/sqrt(d)) v_i restricted to the
 *     tokens of the selected pages, softmax renormalised over them.
 *   - Lemma 1(ii): exact page log-mass s_j(q) = log sum_{i in P_j} exp(q.k_i/sqrt(d)) (the
 *     "exact" arm used as a ceiling and in invariants).
 *
 * Readings taken where the paper is silent (these are all of them):
 *   quantiser = symmetric abs-max, scale = fp16(maxabs/qmax), qmax 7 (int4) / 127 (int8),
 *   code = clamp(rint(x/scale)) round-half-even with the rounded scale; zero-mode threshold
 *   lambda_l <= 1e-6 lambda_1 (or <= 1e-10 of the page's summed squared key norms) and never more
 *   than B-1 modes; eigenvector sign = largest-magnitude
 *   entry positive; shares normalised over the candidate pages 1..P-2 only; ranking by
 *   log m_bar_j, ties to the lower page index; returned ids ascending, -1 padded;
 *   P <= k selects every page.
 *
 * Parity status: every function here, the batch-level wrappers' request / head / block indexing
 * included, is pinned by the CPU tests (closed forms, invariants from the paper's propositions,
 * brute force, numpy cross-checks) EXCEPT the size of the score error
 * caused by the integer storage, for which the paper derives no bound: "parity unpinned" for
 * that one quantity (the integer pack/unpack itself is pinned by round-trip and byte counts).
 *
 * No blocking, fusion or reordering beyond the definitions; loops are written for reading.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORA_F32 0
#define ORA_BF16 1
#define ORA_F64 2

#define ORA_FMT_F32 0
#define ORA_FMT_I4 1
#define ORA_FMT_I8 2   /* int8 basis, int8 coefficients + centroid: the "int8 basis" arm of the paper's precision ablation */
#define ORA_FMT_BF16 3 /* bf16 basis, int8 coefficients + centroid: the paper's "r8fp" control */

typedef struct {
  const void *k, *v;        /* paged cache, element (block, head, token, dim) at
                               block*stride_block + head*stride_head + token*stride_token + dim */
  int32_t dtype;            /* ORA_F32 | ORA_BF16 */
  int64_t stride_block, stride_head, stride_token; /* in elements */
  int32_t num_blocks;
  const int32_t *block_table; /* [batch, max_pages] logical page -> physical block */
  int32_t max_pages;
  const int32_t *seq_lens;    /* [batch] tokens in the sequence */
  int32_t B, d, Hq, Hkv;
} ora_kv;

/* ------------------------------------------------------------------ element access */

static double bf16_to_double(uint16_t h) {
  uint32_t w = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &w, 4);
  return (double)f;
}

static double load_elem(const void *p, int dtype, int64_t idx) {
  if (dtype == ORA_F32) return (double)((const float *)p)[idx];
  if (dtype == ORA_F64) return ((const double *)p)[idx];
  return bf16_to_double(((const uint16_t *)p)[idx]);
}

/* IEEE binary16 <-> double, round to nearest even, written out by hand. */
static double half_to_double(uint16_t h) {
  int sign = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
  double v;
  if (e == 0) v = ldexp((double)m, -24);
  else if (e == 31) v = m ? NAN : INFINITY;
  else v = ldexp((double)(m + 1024), e - 25);
  return sign ? -v : v;
}

static uint16_t double_to_half(double x) {
  uint16_t sign = 0;
  if (x < 0 || (x == 0 && signbit(x))) { sign = 0x8000; x = -x; }
  if (isnan(x)) return (uint16_t)(sign | 0x7e00);
  if (x >= 65520.0) return (uint16_t)(sign | 0x7c00); /* rounds to infinity */
  if (x == 0) return sign;
  int e;
  (void)frexp(x, &e);              /* x = f * 2^e, f in [0.5,1) => exponent of x is e-1 */
  int ex = e - 1;
  if (ex < -14) ex = -14;          /* subnormal range shares the quantum 2^-24 */
  double quantum = ldexp(1.0, ex - 10);
  double n = nearbyint(x / quantum); /* default rounding mode: to nearest, ties to even */
  double r = n * quantum;
  /* re-encode r exactly */
  if (r >= 65520.0) return (uint16_t)(sign | 0x7c00);
  if (r < ldexp(1.0, -14)) return (uint16_t)(sign | (uint16_t)nearbyint(r / ldexp(1.0, -24)));
  (void)frexp(r, &e);
  ex = e - 1;
  uint16_t mant = (uint16_t)(nearbyint(r / ldexp(1.0, ex - 10)) - 1024);
  return (uint16_t)(sign | ((ex + 15) << 10) | mant);
}

uint16_t ora_double_to_half(double x) { return double_to_half(x); }
double ora_half_to_double(uint16_t h) { return half_to_double(h); }

/* ------------------------------------------------------------------ symmetric eigensolver */

/* Cyclic Jacobi on a symmetric n x n matrix A (row-major, overwritten).  On return lam[] holds
 * the eigenvalues in descending order and column l of U (U[i*n+l]) the matching unit
 * eigenvector.  Rotations continue until the off-diagonal Frobenius norm is <= 1e-14 ||A||_F. */
void ora_eigh_jacobi(int n, double *A, double *U, double *lam) {
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) U[i * n + j] = (i == j) ? 1.0 : 0.0;
  double normA = 0;
  for (int i = 0; i < n * n; ++i) normA += A[i] * A[i];
  normA = sqrt(normA);
  for (int sweep = 0; sweep < 100; ++sweep) {
    double off = 0;
    for (int i = 0; i < n; ++i)
      for (int j = 0; j < n; ++j)
        if (i != j) off += A[i * n + j] * A[i * n + j];
    if (sqrt(off) <= 1e-14 * normA || normA == 0) break;
    for (int p = 0; p < n - 1; ++p)
      for (int q = p + 1; q < n; ++q) {
        double apq = A[p * n + q];
        if (apq == 0) continue;
        double theta = (A[q * n + q] - A[p * n + p]) / (2 * apq);
        double t = (theta >= 0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1));
        double c = 1 / sqrt(t * t + 1), s = t * c;
        for (int i = 0; i < n; ++i) { /* A <- A J */
          double aip = A[i * n + p], aiq = A[i * n + q];
          A[i * n + p] = c * aip - s * aiq;
          A[i * n + q] = s * aip + c * aiq;
        }
        for (int i = 0; i < n; ++i) { /* A <- J^T A */
          double api = A[p * n + i], aqi = A[q * n + i];
          A[p * n + i] = c * api - s * aqi;
          A[q * n + i] = s * api + c * aqi;
        }
        for (int i = 0; i < n; ++i) { /* U <- U J */
          double uip = U[i * n + p], uiq = U[i * n + q];
          U[i * n + p] = c * uip - s * uiq;
          U[i * n + q] = s * uip + c * uiq;
        }
      }
  }
  for (int i = 0; i < n; ++i) lam[i] = A[i * n + i];
  /* sort descending (selection sort, columns move with their eigenvalue) */
  for (int a = 0; a < n - 1; ++a) {
    int best = a;
    for (int b = a + 1; b < n; ++b)
      if (lam[b] > lam[best]) best = b;
    if (best != a) {
      double tl = lam[a]; lam[a] = lam[best]; lam[best] = tl;
      for (int i = 0; i < n; ++i) {
        double tu = U[i * n + a]; U[i * n + a] = U[i * n + best]; U[i * n + best] = tu;
      }
    }
  }
}

/* ------------------------------------------------------------------ build (Sec. 4 "Build") */

/* keys: B x d (row i = key of token i).  Outputs: mu[d]; V[l*d + c] (r rows, unit vectors or
 * zero); C[i*r + l]; lam[B] all Gram eigenvalues (descending); returns r_eff. */
int ora_build_page(const double *keys, int B, int d, int r, double *mu, double *V, double *C,
                   double *lam) {
  double *D = (double *)malloc(sizeof(double) * B * d);
  double *M = (double *)malloc(sizeof(double) * B * B);
  double *U = (double *)malloc(sizeof(double) * B * B);
  for (int c = 0; c < d; ++c) {
    double s = 0;
    for (int i = 0; i < B; ++i) s += keys[i * d + c];
    mu[c] = s / B;
  }
  for (int i = 0; i < B; ++i)
    for (int c = 0; c < d; ++c) D[i * d + c] = keys[i * d + c] - mu[c];
  for (int i = 0; i < B; ++i)
    for (int j = 0; j < B; ++j) {
      double s = 0;
      for (int c = 0; c < d; ++c) s += D[i * d + c] * D[j * d + c];
      M[i * B + j] = s;
    }
  ora_eigh_jacobi(B, M, U, lam);
  int rmax = r < B - 1 ? r : B - 1; /* a centred page has at most B-1 nonzero modes */
  int r_eff = 0;
  double knorm2 = 0; /* modes below 1e-10 of the page's key energy are rounding residue of the centring */
  for (int i = 0; i < B * d; ++i) knorm2 += keys[i] * keys[i];
  for (int l = 0; l < rmax; ++l)
    if (lam[0] > 0 && lam[l] > 1e-6 * lam[0] && lam[l] > 1e-10 * knorm2) r_eff = l + 1; else break;
  for (int l = 0; l < r; ++l) {
    if (l < r_eff) {
      double sigma = sqrt(lam[l]);
      for (int c = 0; c < d; ++c) {
        double s = 0;
        for (int i = 0; i < B; ++i) s += D[i * d + c] * U[i * B + l];
        V[l * d + c] = s / sigma;
      }
      for (int i = 0; i < B; ++i) C[i * r + l] = sigma * U[i * B + l];
      /* sign convention: largest-magnitude basis entry positive, lowest index on ties */
      int big = 0;
      for (int c = 1; c < d; ++c)
        if (fabs(V[l * d + c]) > fabs(V[l * d + big])) big = c;
      if (V[l * d + big] < 0) {
        for (int c = 0; c < d; ++c) V[l * d + c] = -V[l * d + c];
        for (int i = 0; i < B; ++i) C[i * r + l] = -C[i * r + l];
      }
    } else {
      for (int c = 0; c < d; ++c) V[l * d + c] = 0;
      for (int i = 0; i < B; ++i) C[i * r + l] = 0;
    }
  }
  free(D); free(M); free(U);
  return r_eff;
}

/* ------------------------------------------------------------------ storage formats */

/* Bytes of one stored summary (what the paper's payload table counts) and its padded stride. */
int64_t ora_summary_payload_bytes(int fmt, int r, int B, int d) {
  if (fmt == ORA_FMT_F32) return 4 * ((int64_t)d + (int64_t)r * d + (int64_t)B * r);
  /* int8 basis d*r, int8 coefficients B*r, int8 centroid d, fp16 scales r + B + 1 */
  if (fmt == ORA_FMT_I8) return (int64_t)d * r + (int64_t)B * r + d + 2 * ((int64_t)r + B + 1);
  /* bf16 basis 2*d*r (no basis scales), int8 coefficients and centroid, fp16 scales B + 1 */
  if (fmt == ORA_FMT_BF16) return 2 * (int64_t)d * r + (int64_t)B * r + d + 2 * ((int64_t)B + 1);
  /* int4 basis d*r/2, int8 coefficients B*r, int8 centroid d, fp16 scales: r + B + 1 */
  return (int64_t)d * r / 2 + (int64_t)B * r + d + 2 * ((int64_t)r + B + 1);
}
int64_t ora_summary_stride_bytes(int fmt, int r, int B, int d) {
  int64_t n = ora_summary_payload_bytes(fmt, r, B, d);
  return (n + 15) / 16 * 16;
}

/* Symmetric abs-max quantiser with an fp16 scale. */
static double quant_scale(const double *x, int n, int stride, int qmax, uint16_t *scale_bits) {
  double m = 0;
  for (int i = 0; i < n; ++i)
    if (fabs(x[i * stride]) > m) m = fabs(x[i * stride]);
  *scale_bits = double_to_half(m / qmax);
  return half_to_double(*scale_bits);
}
static int quant_code(double x, double scale, int qmax) {
  if (scale == 0) return 0;
  double c = nearbyint(x / scale);
  if (c > qmax) c = qmax;
  if (c < -qmax) c = -qmax;
  return (int)c;
}

/* Byte positions of the I4 blob (d a multiple of 16, r in {2,4,8}).
 *   [basis d*r/2][coefficients B r][centroid d][sC B x fp16][sV r x fp16][sMu fp16]
 * Codes are stored offset-binary: nibble = code + 8, byte = code + 128.  The paper fixes the byte COUNT of this
 * format at every page size (App. C.1 payload table, App. D "Page size": 9.4 / 5.5 / 3.5 % of the page's KV bytes at
 * B = 16 / 32 / 64), not the byte order.  Basis and centroid are ordered the same way at every B; coefficients and
 * their scales follow an interleaved order at B = 16 and plain row-major order (token, rank) at other page sizes. */
static void i4_basis_pos(int l, int c, int d, int *byte, int *shift) {
  /* dims are split into 4 contiguous quarters t; inside a quarter, group s covers 4 dims */
  int Q = d / 4, t = c / Q, w = c % Q, s = w >> 2, half = (w >> 1) & 1, e = w & 1;
  int j = s >> 1, i = ((s & 1) << 1) | half, nib = i + 4 * e;
  *byte = (l * 4 + t) * (Q / 2) + j * 4 + (nib >> 1);
  *shift = (nib & 1) * 4;
}
static int i4_coef_pos(int i, int l, int r, int B) {
  if (B != 16) return i * r + l;
  int x = i & 7, hi = i >> 3, tp = l >> 1, e = l & 1;
  return (x * (r / 2) + tp) * 4 + hi * 2 + e;
}
static int i4_mu_pos(int c, int d) {
  int Q = d / 4, t = c / Q, w = c % Q, s = w >> 2, half = (w >> 1) & 1, e = w & 1;
  return t * Q + s * 4 + e * 2 + half;
}
static int i4_sc_pos(int i, int B) {
  if (B != 16) return i;
  int t = (i & 7) >> 1, e = i & 1, hi = i >> 3;
  return t * 4 + hi * 2 + e;
}

void ora_pack(int fmt, int r, int B, int d, const double *mu, const double *V, const double *C,
              uint8_t *blob) {
  int64_t stride = ora_summary_stride_bytes(fmt, r, B, d);
  memset(blob, 0, (size_t)stride);
  if (fmt == ORA_FMT_F32) {
    float *f = (float *)blob;
    for (int c = 0; c < d; ++c) f[c] = (float)mu[c];
    for (int l = 0; l < r; ++l)
      for (int c = 0; c < d; ++c) f[d + l * d + c] = (float)V[l * d + c];
    for (int i = 0; i < B; ++i)
      for (int l = 0; l < r; ++l) f[d + r * d + i * r + l] = (float)C[i * r + l];
    return;
  }
  if (fmt == ORA_FMT_I8 || fmt == ORA_FMT_BF16) {
    /* plain row-major layout: [basis r x d][coefficients B x r][centroid d][sC B][sV r (int8 basis only)][sMu];
       integer codes offset-binary (byte = code + 128), bf16 by round-to-nearest-even */
    int wide = fmt == ORA_FMT_BF16 ? 2 : 1;
    int oc = wide * d * r, om = oc + B * r, osc = om + d, osv = osc + 2 * B, osmu = osv + (fmt == ORA_FMT_I8 ? 2 * r : 0);
    uint16_t hb;
    for (int l = 0; l < r; ++l) {
      if (fmt == ORA_FMT_I8) {
        double sc = quant_scale(V + l * d, d, 1, 127, &hb);
        memcpy(blob + osv + 2 * l, &hb, 2);
        for (int c = 0; c < d; ++c) blob[l * d + c] = (uint8_t)(quant_code(V[l * d + c], sc, 127) + 128);
      } else {
        for (int c = 0; c < d; ++c) {
          float f = (float)V[l * d + c];
          uint32_t u; memcpy(&u, &f, 4);
          uint16_t b16 = (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
          memcpy(blob + 2 * (l * d + c), &b16, 2);
        }
      }
    }
    for (int i = 0; i < B; ++i) {
      double sc = quant_scale(C + i * r, r, 1, 127, &hb);
      memcpy(blob + osc + 2 * i, &hb, 2);
      for (int l = 0; l < r; ++l) blob[oc + i * r + l] = (uint8_t)(quant_code(C[i * r + l], sc, 127) + 128);
    }
    double sc = quant_scale(mu, d, 1, 127, &hb);
    memcpy(blob + osmu, &hb, 2);
    for (int c = 0; c < d; ++c) blob[om + c] = (uint8_t)(quant_code(mu[c], sc, 127) + 128);
    return;
  }
  int off_coef = d * r / 2, off_mu = off_coef + B * r, off_sc = off_mu + d;
  int off_sv = off_sc + 2 * B, off_smu = off_sv + 2 * r;
  uint16_t bits;
  for (int l = 0; l < r; ++l) { /* basis: one scale per column of V (per rank) */
    double sc = quant_scale(V + l * d, d, 1, 7, &bits);
    memcpy(blob + off_sv + 2 * l, &bits, 2);
    for (int c = 0; c < d; ++c) {
      int byte, shift;
      i4_basis_pos(l, c, d, &byte, &shift);
      blob[byte] |= (uint8_t)((quant_code(V[l * d + c], sc, 7) + 8) << shift);
    }
  }
  for (int i = 0; i < B; ++i) { /* coefficients: one scale per row of C (per token) */
    double sc = quant_scale(C + i * r, r, 1, 127, &bits);
    memcpy(blob + off_sc + 2 * i4_sc_pos(i, B), &bits, 2);
    for (int l = 0; l < r; ++l)
      blob[off_coef + i4_coef_pos(i, l, r, B)] = (uint8_t)(quant_code(C[i * r + l], sc, 127) + 128);
  }
  {
    double sc = quant_scale(mu, d, 1, 127, &bits);
    memcpy(blob + off_smu, &bits, 2);
    for (int c = 0; c < d; ++c)
      blob[off_mu + i4_mu_pos(c, d)] = (uint8_t)(quant_code(mu[c], sc, 127) + 128);
  }
}

/* Dequantised stored values, as the scorer sees them. */
void ora_unpack(int fmt, int r, int B, int d, const uint8_t *blob, double *mu, double *V,
                double *C) {
  if (fmt == ORA_FMT_F32) {
    const float *f = (const float *)blob;
    for (int c = 0; c < d; ++c) mu[c] = f[c];
    for (int l = 0; l < r; ++l)
      for (int c = 0; c < d; ++c) V[l * d + c] = f[d + l * d + c];
    for (int i = 0; i < B; ++i)
      for (int l = 0; l < r; ++l) C[i * r + l] = f[d + r * d + i * r + l];
    return;
  }
  if (fmt == ORA_FMT_I8 || fmt == ORA_FMT_BF16) {
    int wide = fmt == ORA_FMT_BF16 ? 2 : 1;
    int oc = wide * d * r, om = oc + B * r, osc = om + d, osv = osc + 2 * B, osmu = osv + (fmt == ORA_FMT_I8 ? 2 * r : 0);
    uint16_t hb;
    for (int l = 0; l < r; ++l) {
      double sc = 1;
      if (fmt == ORA_FMT_I8) { memcpy(&hb, blob + osv + 2 * l, 2); sc = half_to_double(hb); }
      for (int c = 0; c < d; ++c) {
        if (fmt == ORA_FMT_I8) V[l * d + c] = sc * ((int)blob[l * d + c] - 128);
        else {
          uint16_t b16; memcpy(&b16, blob + 2 * (l * d + c), 2);
          uint32_t u = (uint32_t)b16 << 16; float f; memcpy(&f, &u, 4);
          V[l * d + c] = f;
        }
      }
    }
    for (int i = 0; i < B; ++i) {
      memcpy(&hb, blob + osc + 2 * i, 2);
      double sc = half_to_double(hb);
      for (int l = 0; l < r; ++l) C[i * r + l] = sc * ((int)blob[oc + i * r + l] - 128);
    }
    memcpy(&hb, blob + osmu, 2);
    double sc = half_to_double(hb);
    for (int c = 0; c < d; ++c) mu[c] = sc * ((int)blob[om + c] - 128);
    return;
  }
  int off_coef = d * r / 2, off_mu = off_coef + B * r, off_sc = off_mu + d;
  int off_sv = off_sc + 2 * B, off_smu = off_sv + 2 * r;
  uint16_t bits;
  for (int l = 0; l < r; ++l) {
    memcpy(&bits, blob + off_sv + 2 * l, 2);
    double sc = half_to_double(bits);
    for (int c = 0; c < d; ++c) {
      int byte, shift;
      i4_basis_pos(l, c, d, &byte, &shift);
      V[l * d + c] = sc * (((blob[byte] >> shift) & 15) - 8);
    }
  }
  for (int i = 0; i < B; ++i) {
    memcpy(&bits, blob + off_sc + 2 * i4_sc_pos(i, B), 2);
    double sc = half_to_double(bits);
    for (int l = 0; l < r; ++l) C[i * r + l] = sc * ((int)blob[off_coef + i4_coef_pos(i, l, r, B)] - 128);
  }
  memcpy(&bits, blob + off_smu, 2);
  double sc = half_to_double(bits);
  for (int c = 0; c < d; ++c) mu[c] = sc * ((int)blob[off_mu + i4_mu_pos(c, d)] - 128);
}

/* Raw integer codes of an I4 blob (for code-agreement checks): codesV[l*d+c], codesC[i*r+l],
 * codesMu[c], scales as doubles sV[r], sC[B], sMu[1]. */
void ora_unpack_codes(int r, int B, int d, const uint8_t *blob, int32_t *cV, int32_t *cC,
                      int32_t *cMu, double *sV, double *sC, double *sMu) {
  int off_coef = d * r / 2, off_mu = off_coef + B * r, off_sc = off_mu + d;
  int off_sv = off_sc + 2 * B, off_smu = off_sv + 2 * r;
  uint16_t bits;
  for (int l = 0; l < r; ++l) {
    memcpy(&bits, blob + off_sv + 2 * l, 2);
    sV[l] = half_to_double(bits);
    for (int c = 0; c < d; ++c) {
      int byte, shift;
      i4_basis_pos(l, c, d, &byte, &shift);
      cV[l * d + c] = ((blob[byte] >> shift) & 15) - 8;
    }
  }
  for (int i = 0; i < B; ++i) {
    memcpy(&bits, blob + off_sc + 2 * i4_sc_pos(i, B), 2);
    sC[i] = half_to_double(bits);
    for (int l = 0; l < r; ++l) cC[i * r + l] = (int)blob[off_coef + i4_coef_pos(i, l, r, B)] - 128;
  }
  memcpy(&bits, blob + off_smu, 2);
  *sMu = half_to_double(bits);
  for (int c = 0; c < d; ++c) cMu[c] = (int)blob[off_mu + i4_mu_pos(c, d)] - 128;
}

/* ------------------------------------------------------------------ score, Eq. (1) */

double ora_score(int B, int d, int r, const double *mu, const double *V, const double *C,
                 const double *q, double sm_scale) {
  double p[64];
  for (int l = 0; l < r; ++l) {
    double s = 0;
    for (int c = 0; c < d; ++c) s += V[l * d + c] * q[c];
    p[l] = s;
  }
  double a = 0;
  for (int c = 0; c < d; ++c) a += mu[c] * q[c];
  double logit[1024], mx = -INFINITY;
  for (int i = 0; i < B; ++i) {
    double s = a;
    for (int l = 0; l < r; ++l) s += p[l] * C[i * r + l];
    logit[i] = sm_scale * s;
    if (logit[i] > mx) mx = logit[i];
  }
  double z = 0;
  for (int i = 0; i < B; ++i) z += exp(logit[i] - mx);
  return mx + log(z);
}

/* Rival page scores the paper measures the summary against (App. A / App. B), from the same summary:
 *   scorer 1, centroid only:  q.mu/sqrt(d) + log B
 *   scorer 2, rank-r moment core (Eq. 3): q.mu/sqrt(d) + log B + (1/(2 B d)) sum_{l<=r} sigma_l^2 (v_l.q)^2.
 *             With z_i = (V^T q).c_i / sqrt(d) the reconstructed within-page logits, sum_i z_i^2 equals
 *             (1/d) sum_l sigma_l^2 (v_l.q)^2 because the columns of C = U_r Sigma_r are orthogonal with squared
 *             norms sigma_l^2; the score is evaluated in that form, (1/(2B)) sum_i z_i^2, so that it is defined
 *             by the stored (possibly quantised) values alone. */
double ora_rival_score(int scorer, int B, int d, int r, const double *mu, const double *V, const double *C,
                       const double *q, double sm_scale) {
  double a = 0;
  for (int c = 0; c < d; ++c) a += mu[c] * q[c];
  double s = sm_scale * a + log((double)B);
  if (scorer == 2) {
    double *p = (double *)malloc(sizeof(double) * r);
    for (int l = 0; l < r; ++l) {
      p[l] = 0;
      for (int c = 0; c < d; ++c) p[l] += V[l * d + c] * q[c];
    }
    double z2 = 0;
    for (int i = 0; i < B; ++i) {
      double z = 0;
      for (int l = 0; l < r; ++l) z += p[l] * C[i * r + l];
      z2 += (sm_scale * z) * (sm_scale * z);
    }
    s += z2 / (2.0 * B);
    free(p);
  }
  return s;
}

/* The min/max envelope score (Lemma 2): sum_c max(q_c u_c, q_c l_c) * sm_scale over the first ntok keys. */
double ora_envelope_score(int ntok, int d, const double *keys, const double *q, double sm_scale) {
  double e = 0;
  for (int c = 0; c < d; ++c) {
    double u = -INFINITY, l = INFINITY;
    for (int i = 0; i < ntok; ++i) {
      if (keys[i * d + c] > u) u = keys[i * d + c];
      if (keys[i * d + c] < l) l = keys[i * d + c];
    }
    e += (q[c] * u > q[c] * l) ? q[c] * u : q[c] * l;
  }
  return sm_scale * e;
}

/* exact page log-mass of Lemma 1(ii) over the first ntok keys (rows of keys, ntok x d) */
double ora_exact_lse(int ntok, int d, const double *keys, const double *q, double sm_scale) {
  double mx = -INFINITY, logit[1024];
  for (int i = 0; i < ntok; ++i) {
    double s = 0;
    for (int c = 0; c < d; ++c) s += keys[i * d + c] * q[c];
    logit[i] = sm_scale * s;
    if (logit[i] > mx) mx = logit[i];
  }
  double z = 0;
  for (int i = 0; i < ntok; ++i) z += exp(logit[i] - mx);
  return mx + log(z);
}

/* ------------------------------------------------------------------ batch-level steps */

static int g_threads = 1;
void ora_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int ora_get_max_threads(void) {
#ifdef _OPENMP
  return omp_get_num_procs();
#else
  return 1;
#endif
}

static int num_pages(int T, int B) { return (T + B - 1) / B; }

static void load_page_keys(const ora_kv *kv, const void *base, int block, int h, int ntok,
                           double *out) {
  for (int i = 0; i < ntok; ++i)
    for (int c = 0; c < kv->d; ++c)
      out[i * kv->d + c] = load_elem(base, kv->dtype,
          (int64_t)block * kv->stride_block + (int64_t)h * kv->stride_head +
          (int64_t)i * kv->stride_token + c);
}

/* Build the summary of every COMPLETE page p with page_begin[b] <= p < page_end[b] (NULL, NULL =
 * all complete pages) of every request and KV head; blob (block, head) lives at
 * summaries + (block*Hkv + head)*stride. */
void ora_build_summaries(const ora_kv *kv, int batch, int r, int fmt, const int32_t *page_begin,
                         const int32_t *page_end, uint8_t *summaries) {
  int B = kv->B, d = kv->d;
  int64_t stride = ora_summary_stride_bytes(fmt, r, B, d);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int h = 0; h < kv->Hkv; ++h) {
      int complete = kv->seq_lens[b] / B;
      int p0 = page_begin ? page_begin[b] : 0, p1 = page_end ? page_end[b] : complete;
      if (p1 > complete) p1 = complete;
      double *keys = (double *)malloc(sizeof(double) * B * d);
      double *mu = (double *)malloc(sizeof(double) * d);
      double *V = (double *)malloc(sizeof(double) * r * d);
      double *C = (double *)malloc(sizeof(double) * B * r);
      double *lam = (double *)malloc(sizeof(double) * B);
      for (int p = p0; p < p1; ++p) {
        int block = kv->block_table[(int64_t)b * kv->max_pages + p];
        load_page_keys(kv, kv->k, block, h, B, keys);
        ora_build_page(keys, B, d, r, mu, V, C, lam);
        ora_pack(fmt, r, B, d, mu, V, C, summaries + ((int64_t)block * kv->Hkv + h) * stride);
      }
      free(keys); free(mu); free(V); free(C); free(lam);
    }
}

/* Estimated (exact = 0) or exact (exact = 1) page log-mass of every complete page below the last
 * one: shat[(b*Hq + g)*max_pages + p] for p in [0, P-1) ; other entries are left untouched. */
void ora_page_logmass(const ora_kv *kv, int batch, const void *q, int q_dtype, int r, int fmt,
                      const uint8_t *summaries, double sm_scale, int exact, double *shat) {
  int B = kv->B, d = kv->d, G = kv->Hq / kv->Hkv;
  int64_t stride = ora_summary_stride_bytes(fmt, r, B, d);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int h = 0; h < kv->Hkv; ++h) {
      int P = num_pages(kv->seq_lens[b], B);
      double *keys = (double *)malloc(sizeof(double) * B * d);
      double *mu = (double *)malloc(sizeof(double) * d);
      double *V = (double *)malloc(sizeof(double) * r * d);
      double *C = (double *)malloc(sizeof(double) * B * r);
      double *qd = (double *)malloc(sizeof(double) * d);
      for (int p = 0; p < P - 1; ++p) {
        int block = kv->block_table[(int64_t)b * kv->max_pages + p];
        if (exact) load_page_keys(kv, kv->k, block, h, B, keys);
        else ora_unpack(fmt, r, B, d, summaries + ((int64_t)block * kv->Hkv + h) * stride, mu, V, C);
        for (int gi = 0; gi < G; ++gi) {
          int g = h * G + gi;
          for (int c = 0; c < d; ++c) qd[c] = load_elem(q, q_dtype, ((int64_t)b * kv->Hq + g) * d + c);
          shat[((int64_t)b * kv->Hq + g) * kv->max_pages + p] =
              exact ? ora_exact_lse(B, d, keys, qd, sm_scale)
                    : ora_score(B, d, r, mu, V, C, qd, sm_scale);
        }
      }
      free(keys); free(mu); free(V); free(C); free(qd);
    }
}

/* KIVI-style fake quantisation of complete pages, in place (Sec. 5; App. C protocol): keys per channel over the
 * page's B tokens, values per token over groups of 32 dims; asymmetric uniform grid of 2^bits levels between the
 * group's minimum and maximum, x^ = min + s rint((x - min)/s), s = (max - min)/(2^bits - 1); a constant group is
 * kept.  The result is stored back in the cache's element type (round to nearest even for bf16).  k, v must be
 * writable.  Only fp32 and bf16 caches. */
static void store_elem(void *base, int dtype, int64_t idx, double x) {
  if (dtype == ORA_F32) { ((float *)base)[idx] = (float)x; return; }
  float f = (float)x;
  uint32_t u; memcpy(&u, &f, 4);
  uint32_t r = u + 0x7FFFu + ((u >> 16) & 1u);   /* round to nearest even on the dropped 16 bits */
  ((uint16_t *)base)[idx] = (uint16_t)(r >> 16);
}
static double requant(double x, double lo, double hi, int levels) {
  double s = (hi - lo) / levels;
  if (!(s > 0)) return x;
  return lo + s * rint((x - lo) / s);
}
void ora_fake_quantize_pages(const ora_kv *kv, int batch, const int32_t *page_begin, const int32_t *page_end, int bits) {
  int B = kv->B, d = kv->d, levels = (1 << bits) - 1;
  for (int b = 0; b < batch; ++b)
    for (int h = 0; h < kv->Hkv; ++h) {
      int complete = kv->seq_lens[b] / B;
      int p0 = page_begin ? page_begin[b] : 0, p1 = page_end ? page_end[b] : complete;
      if (p1 > complete) p1 = complete;
      for (int p = p0; p < p1; ++p) {
        int block = kv->block_table[(int64_t)b * kv->max_pages + p];
        int64_t base = (int64_t)block * kv->stride_block + (int64_t)h * kv->stride_head;
        for (int c = 0; c < d; ++c) { /* keys: one group per channel */
          double lo = INFINITY, hi = -INFINITY;
          for (int i = 0; i < B; ++i) {
            double x = load_elem(kv->k, kv->dtype, base + (int64_t)i * kv->stride_token + c);
            if (x < lo) lo = x;
            if (x > hi) hi = x;
          }
          for (int i = 0; i < B; ++i) {
            int64_t at = base + (int64_t)i * kv->stride_token + c;
            store_elem((void *)kv->k, kv->dtype, at, requant(load_elem(kv->k, kv->dtype, at), lo, hi, levels));
          }
        }
        for (int i = 0; i < B; ++i) /* values: groups of 32 dims of one token */
          for (int g0 = 0; g0 < d; g0 += 32) {
            double lo = INFINITY, hi = -INFINITY;
            for (int c = g0; c < g0 + 32 && c < d; ++c) {
              double x = load_elem(kv->v, kv->dtype, base + (int64_t)i * kv->stride_token + c);
              if (x < lo) lo = x;
              if (x > hi) hi = x;
            }
            for (int c = g0; c < g0 + 32 && c < d; ++c) {
              int64_t at = base + (int64_t)i * kv->stride_token + c;
              store_elem((void *)kv->v, kv->dtype, at, requant(load_elem(kv->v, kv->dtype, at), lo, hi, levels));
            }
          }
      }
    }
}

/* Rival scores of every page (scorer 1, 2: pages 0..P-2 from the summaries; scorer 3, envelope: pages 0..P-1 from
 * the keys): out[(b*Hq + g)*max_pages + p]. */
void ora_rival_logmass(const ora_kv *kv, int batch, const void *q, int q_dtype, int r, int fmt,
                       const uint8_t *summaries, double sm_scale, int scorer, double *out) {
  int B = kv->B, d = kv->d, G = kv->Hq / kv->Hkv;
  int64_t stride = ora_summary_stride_bytes(fmt, r, B, d);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int h = 0; h < kv->Hkv; ++h) {
      int T = kv->seq_lens[b], P = num_pages(T, B);
      double *keys = (double *)malloc(sizeof(double) * B * d);
      double *mu = (double *)malloc(sizeof(double) * d);
      double *V = (double *)malloc(sizeof(double) * r * d);
      double *C = (double *)malloc(sizeof(double) * B * r);
      double *qd = (double *)malloc(sizeof(double) * d);
      int last = scorer == 3 ? P : P - 1;
      for (int p = 0; p < last; ++p) {
        int block = kv->block_table[(int64_t)b * kv->max_pages + p];
        int ntok = T - p * B < B ? T - p * B : B;
        if (scorer == 3) load_page_keys(kv, kv->k, block, h, ntok, keys);
        else ora_unpack(fmt, r, B, d, summaries + ((int64_t)block * kv->Hkv + h) * stride, mu, V, C);
        for (int gi = 0; gi < G; ++gi) {
          int g = h * G + gi;
          for (int c = 0; c < d; ++c) qd[c] = load_elem(q, q_dtype, ((int64_t)b * kv->Hq + g) * d + c);
          out[((int64_t)b * kv->Hq + g) * kv->max_pages + p] =
              scorer == 3 ? ora_envelope_score(ntok, d, keys, qd, sm_scale)
                          : ora_rival_score(scorer, B, d, r, mu, V, C, qd, sm_scale);
        }
      }
      free(keys); free(mu); free(V); free(C); free(qd);
    }
}

/* Share-average combine + budgeted selection for one KV head of one request.
 * s: G rows of page scores with row stride ld (entries 1..P-2 are read).  logshare (optional,
 * length >= P): log m_bar_j for candidates, untouched elsewhere.  ids: k entries. */
int ora_select_one(int P, int G, int k, const double *s, int64_t ld, int32_t *ids, double *logshare) {
  if (P <= k) {
    for (int j = 0; j < k; ++j) ids[j] = j < P ? j : -1;
    return P;
  }
  int ncand = P - 2;
  double *logm = (double *)malloc(sizeof(double) * P);
  double *logZ = (double *)malloc(sizeof(double) * G);
  char *taken = (char *)calloc(P, 1);
  for (int g = 0; g < G; ++g) { /* partition function over the candidate pages */
    double mx = -INFINITY, z = 0;
    for (int j = 1; j <= ncand; ++j) if (s[g * ld + j] > mx) mx = s[g * ld + j];
    for (int j = 1; j <= ncand; ++j) z += exp(s[g * ld + j] - mx);
    logZ[g] = mx + log(z);
  }
  for (int j = 1; j <= ncand; ++j) { /* log of the group-averaged share */
    double mx = -INFINITY, z = 0;
    for (int g = 0; g < G; ++g) if (s[g * ld + j] - logZ[g] > mx) mx = s[g * ld + j] - logZ[g];
    for (int g = 0; g < G; ++g) z += exp(s[g * ld + j] - logZ[g] - mx);
    logm[j] = mx + log(z) - log((double)G);
    if (logshare) logshare[j] = logm[j];
  }
  taken[0] = 1; taken[P - 1] = 1; /* sink and most recent page */
  for (int n = 0; n < k - 2; ++n) { /* repeated arg-max, ties to the lower index */
    int best = -1;
    for (int j = 1; j <= ncand; ++j)
      if (!taken[j] && (best < 0 || logm[j] > logm[best])) best = j;
    taken[best] = 1;
  }
  int cnt = 0;
  for (int j = 0; j < P; ++j) if (taken[j]) ids[cnt++] = j;
  free(logm); free(logZ); free(taken);
  return cnt;
}

/* The combine rules the paper ablates against its own (App. D, GQA combine table), same selection otherwise:
 * rule 0 share-average (ora_select_one), rule 1 group-max: key_j = max_g s_j(q_g), rule 2 group-mass:
 * key_j = log sum_g exp s_j(q_g).  key (optional, length >= P) receives the ranking key of the candidates. */
int ora_select_one_rule(int P, int G, int k, const double *s, int64_t ld, int rule, int32_t *ids, double *key) {
  if (rule == 0) return ora_select_one(P, G, k, s, ld, ids, key);
  if (P <= k) {
    for (int j = 0; j < k; ++j) ids[j] = j < P ? j : -1;
    return P;
  }
  double *kk = (double *)malloc(sizeof(double) * P);
  char *taken = (char *)calloc(P, 1);
  for (int j = 1; j <= P - 2; ++j) {
    double mx = -INFINITY, z = 0;
    for (int g = 0; g < G; ++g) if (s[g * ld + j] > mx) mx = s[g * ld + j];
    for (int g = 0; g < G; ++g) z += exp(s[g * ld + j] - mx);
    kk[j] = rule == 1 ? mx : mx + log(z);
    if (key) key[j] = kk[j];
  }
  taken[0] = 1; taken[P - 1] = 1;
  for (int n = 0; n < k - 2; ++n) {
    int best = -1;
    for (int j = 1; j <= P - 2; ++j)
      if (!taken[j] && (best < 0 || kk[j] > kk[best])) best = j;
    taken[best] = 1;
  }
  int cnt = 0;
  for (int j = 0; j < P; ++j) if (taken[j]) ids[cnt++] = j;
  free(kk); free(taken);
  return cnt;
}

void ora_select(const ora_kv *kv, int batch, int k, const double *shat, int32_t *page_ids,
                int32_t *page_count, double *logshare) {
  int G = kv->Hq / kv->Hkv;
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int h = 0; h < kv->Hkv; ++h) {
      int P = num_pages(kv->seq_lens[b], kv->B);
      int64_t prob = (int64_t)b * kv->Hkv + h;
      page_count[prob] = ora_select_one(P, G, k, shat + ((int64_t)b * kv->Hq + h * G) * kv->max_pages,
                                        kv->max_pages, page_ids + prob * k,
                                        logshare ? logshare + prob * kv->max_pages : NULL);
    }
}
/* Per-head arm: every query head ranks the pages by its own share and keeps its own k pages (a group of one):
 * page_ids [batch][Hq][k], page_count [batch][Hq], logshare [batch][Hq][max_pages] = log share of the head. */
void ora_select_per_head(const ora_kv *kv, int batch, int k, const double *shat, int32_t *page_ids,
                         int32_t *page_count, double *logshare) {
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int g = 0; g < kv->Hq; ++g) {
      int P = num_pages(kv->seq_lens[b], kv->B);
      int64_t row = (int64_t)b * kv->Hq + g;
      page_count[row] = ora_select_one(P, 1, k, shat + row * kv->max_pages, kv->max_pages, page_ids + row * k,
                                       logshare ? logshare + row * kv->max_pages : NULL);
    }
}

/* Softmax attention of every query head over the tokens (< T) of the listed pages.
 * page_ids == NULL: every page (dense attention).  out[(b*Hq+g)*d + c], lse[b*Hq+g]. */
/* per_head = 0: one page table per (request, KV head), shared by the group's query heads (the method);
 * per_head = 1: one page table per (request, query head) (the per-head arm of App. D's combine table). */
static void attend_impl(const ora_kv *kv, int batch, const void *q, int q_dtype, double sm_scale, int k,
                        const int32_t *page_ids, const int32_t *page_count, double *out, double *lse, int per_head) {
  int B = kv->B, d = kv->d, G = kv->Hq / kv->Hkv;
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int g = 0; g < kv->Hq; ++g) {
      int h = g / G, T = kv->seq_lens[b], P = num_pages(T, B);
      int64_t prob = per_head ? (int64_t)b * kv->Hq + g : (int64_t)b * kv->Hkv + h;
      int npages = page_ids ? page_count[prob] : P;
      double *qd = (double *)malloc(sizeof(double) * d);
      double *x = (double *)malloc(sizeof(double) * (size_t)npages * B);
      int *tokpage = (int *)malloc(sizeof(int) * (size_t)npages * B);
      int *tokslot = (int *)malloc(sizeof(int) * (size_t)npages * B);
      for (int c = 0; c < d; ++c) qd[c] = load_elem(q, q_dtype, ((int64_t)b * kv->Hq + g) * d + c);
      int n = 0;
      double mx = -INFINITY;
      for (int jj = 0; jj < npages; ++jj) {
        int p = page_ids ? page_ids[prob * k + jj] : jj;
        int block = kv->block_table[(int64_t)b * kv->max_pages + p];
        for (int i = 0; i < B && p * B + i < T; ++i) {
          double s = 0;
          for (int c = 0; c < d; ++c)
            s += qd[c] * load_elem(kv->k, kv->dtype, (int64_t)block * kv->stride_block +
                                   (int64_t)h * kv->stride_head + (int64_t)i * kv->stride_token + c);
          x[n] = sm_scale * s; tokpage[n] = block; tokslot[n] = i;
          if (x[n] > mx) mx = x[n];
          ++n;
        }
      }
      double z = 0;
      for (int i = 0; i < n; ++i) z += exp(x[i] - mx);
      for (int c = 0; c < d; ++c) {
        double acc = 0;
        for (int i = 0; i < n; ++i)
          acc += exp(x[i] - mx) * load_elem(kv->v, kv->dtype, (int64_t)tokpage[i] * kv->stride_block +
                     (int64_t)h * kv->stride_head + (int64_t)tokslot[i] * kv->stride_token + c);
        out[((int64_t)b * kv->Hq + g) * d + c] = acc / z;
      }
      if (lse) lse[(int64_t)b * kv->Hq + g] = mx + log(z);
      free(qd); free(x); free(tokpage); free(tokslot);
    }
}
void ora_attend(const ora_kv *kv, int batch, const void *q, int q_dtype, double sm_scale, int k,
                const int32_t *page_ids, const int32_t *page_count, double *out, double *lse) {
  attend_impl(kv, batch, q, q_dtype, sm_scale, k, page_ids, page_count, out, lse, 0);
}
/* Per-head arm (App. D, GQA combine table, "per-head" row): page_ids [batch][Hq][k], page_count [batch][Hq]. */
void ora_attend_per_head(const ora_kv *kv, int batch, const void *q, int q_dtype, double sm_scale, int k,
                         const int32_t *page_ids, const int32_t *page_count, double *out, double *lse) {
  attend_impl(kv, batch, q, q_dtype, sm_scale, k, page_ids, page_count, out, lse, 1);
}

/* Exact log-mass of EVERY page 0..P-1 (the last page over its valid tokens), Lemma 1(ii):
 * mass[(b*Hq + g)*max_pages + p].  Other entries are left untouched. */
void ora_page_exact_mass_all(const ora_kv *kv, int batch, const void *q, int q_dtype, double sm_scale,
                             double *mass) {
  int B = kv->B, d = kv->d, G = kv->Hq / kv->Hkv;
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    for (int h = 0; h < kv->Hkv; ++h) {
      int T = kv->seq_lens[b], P = num_pages(T, B);
      double *keys = (double *)malloc(sizeof(double) * B * d);
      double *qd = (double *)malloc(sizeof(double) * d);
      for (int p = 0; p < P; ++p) {
        int ntok = T - p * B < B ? T - p * B : B;
        int block = kv->block_table[(int64_t)b * kv->max_pages + p];
        load_page_keys(kv, kv->k, block, h, ntok, keys);
        for (int gi = 0; gi < G; ++gi) {
          int g = h * G + gi;
          for (int c = 0; c < d; ++c) qd[c] = load_elem(q, q_dtype, ((int64_t)b * kv->Hq + g) * d + c);
          mass[((int64_t)b * kv->Hq + g) * kv->max_pages + p] = ora_exact_lse(ntok, d, keys, qd, sm_scale);
        }
      }
      free(keys); free(qd);
    }
}

/* Selection fidelity of a page set A against exact page log-masses (App. B, selection-fidelity table), for one
 * KV head of one request, averaged over its G query heads.  s: G rows (stride ld) of exact log-masses of pages
 * 0..P-1.  A / R: page lists of the table under test / of the reference ranking.  marked: pages of interest
 * ("carriers"; entries outside 1..P-2 are ignored).
 *   out[0] gamma   = sum_{j in A} e^{s_j} / sum_{j<P} e^{s_j}
 *   out[1] gamma_c = the same with pages 0 and P-1 removed from numerator and denominator
 *   out[2] recall  = |A n R| / |R| counted over candidate pages 1..P-2
 *   out[3] needle  = |marked n R n A| / |marked n R|
 * An empty denominator reads 1. */
void ora_selection_quality(int P, int G, const double *s, int64_t ld, const int32_t *A, int na,
                           const int32_t *R, int nr, const int32_t *marked, int nm, double *out) {
  double gam = 0, gamc = 0;
  for (int g = 0; g < G; ++g) {
    const double *sg = s + g * ld;
    double mx = -INFINITY, z = 0, kept = 0, always;
    for (int j = 0; j < P; ++j) if (sg[j] > mx) mx = sg[j];
    for (int j = 0; j < P; ++j) z += exp(sg[j] - mx);
    for (int i = 0; i < na; ++i) if (A[i] >= 0 && A[i] < P) kept += exp(sg[A[i]] - mx);
    always = exp(sg[0] - mx) + (P > 1 ? exp(sg[P - 1] - mx) : 0.0);
    gam += kept / z;
    gamc += (z - always > 0) ? (kept - always > 0 ? kept - always : 0.0) / (z - always) : 1.0;
  }
  out[0] = gam / G;
  out[1] = gamc / G;
  int hit = 0, tot = 0, nk = 0, nh = 0;
  for (int j = 0; j < nr; ++j) {
    if (R[j] <= 0 || R[j] >= P - 1) continue;
    ++tot;
    for (int i = 0; i < na; ++i) if (A[i] == R[j]) { ++hit; break; }
  }
  for (int j = 0; j < nm; ++j) {
    int in_r = 0, in_a = 0;
    if (marked[j] <= 0 || marked[j] >= P - 1) continue;
    for (int i = 0; i < nr; ++i) in_r |= R[i] == marked[j];
    for (int i = 0; i < na; ++i) in_a |= A[i] == marked[j];
    if (in_r) { ++nk; nh += in_a; }
  }
  out[2] = tot ? (double)hit / tot : 1.0;
  out[3] = nk ? (double)nh / nk : 1.0;
}

/* One decode step on resident summaries: score -> select -> attend (the timed CPU baseline).
 * shat is caller-provided scratch [batch, Hq, max_pages]. */
void ora_decode_step(const ora_kv *kv, int batch, const void *q, int q_dtype, int r, int fmt,
                     const uint8_t *summaries, double sm_scale, int k, double *shat,
                     int32_t *page_ids, int32_t *page_count, double *out, double *lse) {
  ora_page_logmass(kv, batch, q, q_dtype, r, fmt, summaries, sm_scale, 0, shat);
  ora_select(kv, batch, k, shat, page_ids, page_count, NULL);
  ora_attend(kv, batch, q, q_dtype, sm_scale, k, page_ids, page_count, out, lse);
}
