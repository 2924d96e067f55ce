// KV-cache fake-quantisation of finalised pages (Sec. 5 "KV-cache quantization under extreme sparsity"; App. C
// KIVI grid): quantise-dequantise in place, in the cache's own element type, so that the attention and build
// kernels run unchanged on the quantised values.  KIVI's grouping, page-aligned as in the paper's protocol:
//   keys    per channel: one group = the 16 tokens of the page in one dimension (per-channel quantisation along
//           the token axis);
//   values  per token: groups of 32 consecutive dimensions of one token;
// asymmetric uniform grid of 2^bits levels between the group's minimum and maximum:
//   s = (max - min) / (2^bits - 1),  x^ = min + s * rint((x - min) / s)   (s = 0: the group is constant, kept).
// "post" = summaries built from the original keys, then this; "pre" = this, then the build: the two arms of the
// paper's grid are two call orders.  The partial last page of a sequence is never touched.
#include "locks_internal.cuh"

namespace {

struct QuantParams {
  void *k, *v;
  int64_t sb, sh, st;
  const int32_t *block_table, *seq_lens, *page_begin, *page_end;
  int32_t *status;
  int Hkv, Pmax, num_blocks, levels;   // levels = 2^bits - 1
};

__device__ __forceinline__ float requant(float x, float lo, float scale, float inv) {
  return scale == 0.f ? x : fmaf(rintf((x - lo) * inv), scale, lo);
}

// one warp per (page, KV head); a lane owns four consecutive dims
template <typename T>
__global__ void __launch_bounds__(128) fake_quant_kernel(QuantParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int h = blockIdx.y, b = blockIdx.z;
  const int complete = p.seq_lens[b] / LOCKS_B;
  const int p0 = p.page_begin ? p.page_begin[b] : 0;
  const int p1 = min(p.page_end ? p.page_end[b] : complete, complete);
  const int page = p0 + blockIdx.x * 4 + warp;
  if (page < 0 || page >= p1 || page >= p.Pmax) return;
  const int block = p.block_table[(int64_t)b * p.Pmax + page];
  if (block < 0 || block >= p.num_blocks) {
    if (lane == 0) set_status(p.status, LOCKS_ERR_BAD_BLOCK);
    return;
  }
  const int64_t base = (int64_t)block * p.sb + (int64_t)h * p.sh + lane * 4;
  T *K = reinterpret_cast<T *>(p.k), *V = reinterpret_cast<T *>(p.v);
  const float nl = (float)p.levels;
  // keys: per channel over the page's tokens
  {
    float x[LOCKS_B][4], lo[4], hi[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) { lo[u] = INFINITY; hi[u] = -INFINITY; }
#pragma unroll
    for (int i = 0; i < LOCKS_B; ++i)
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        x[i][u] = ldf<T>(K, base + (int64_t)i * p.st + u);
        lo[u] = fminf(lo[u], x[i][u]); hi[u] = fmaxf(hi[u], x[i][u]);
      }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float scale = (hi[u] - lo[u]) / nl, inv = scale > 0.f ? 1.f / scale : 0.f;
#pragma unroll
      for (int i = 0; i < LOCKS_B; ++i) stf<T>(K, base + (int64_t)i * p.st + u, requant(x[i][u], lo[u], scale, inv));
    }
  }
  // values: per token over groups of 32 dims = 8 lanes
#pragma unroll 4
  for (int i = 0; i < LOCKS_B; ++i) {
    float x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) x[u] = ldf<T>(V, base + (int64_t)i * p.st + u);
    float lo = fminf(fminf(x[0], x[1]), fminf(x[2], x[3])), hi = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    const float scale = (hi - lo) / nl, inv = scale > 0.f ? 1.f / scale : 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) stf<T>(V, base + (int64_t)i * p.st + u, requant(x[u], lo, scale, inv));
  }
}

}  // namespace

int locks_launch_fake_quant(locks_ctx *c, const locks_kv *kv, int batch, const int32_t *pb, const int32_t *pe, int bits,
                            cudaStream_t st) {
  QuantParams p;
  p.k = kv->k; p.v = kv->v; p.sb = kv->stride_block; p.sh = kv->stride_head; p.st = kv->stride_token;
  p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.page_begin = pb; p.page_end = pe; p.status = c->status;
  p.Hkv = c->cfg.num_kv_heads; p.Pmax = c->Pmax; p.num_blocks = kv->num_blocks; p.levels = (1 << bits) - 1;
  dim3 grid((c->Pmax + 3) / 4, p.Hkv, batch);
  if (c->cfg.kv_dtype == LOCKS_BF16) fake_quant_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>(p);
  else fake_quant_kernel<float><<<grid, 128, 0, st>>>(p);
  return locks_check_launch(c);
}
