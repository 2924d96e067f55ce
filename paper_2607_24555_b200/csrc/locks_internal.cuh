// Internal declarations of liblocks: context, workspace partition, device helpers, launchers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "locks.h"

#define LOCKS_D 128          // head dimension the kernels are written for
#define LOCKS_B 16           // tokens per page of the main (tensor-core) paths; pages of 32 and 64 tokens
                             // (cfg.page_size) go through the plain fp32 kernels, which take the size at run time
#define LOCKS_GROUP 8        // pages scored together by one warp in the scan (one ring stage, one partial)
#define LOCKS_SEL_THREADS 512
#define LOCKS_SEL_MAX_EPT 16 // pages per thread a selector CTA ranks at most (512 threads: 8192 pages or list entries)
#define LOCKS_ATT_WARPS 3        // warps per attend CTA
#define LOCKS_ATT_STAGES 2       // pages (4 KB of K + 4 KB of V each) in each warp's ring
#define LOCKS_ATT_CTAS_PER_SM 4  // 4 x 48 KB of shared memory
#define LOCKS_ATT_MAX_SPLITS 128
#define LOCKS_ATT_SLOT_BOUND 1024 // upper bound on resident attend CTAs of any supported GPU (148 SMs x 4 on B200)
#ifndef LOCKS_SCAN_GATHER
#define LOCKS_SCAN_GATHER 1    // tensor scan: stage summaries four at a time with tensor-map gathers
#endif
#ifndef LOCKS_SCAN_BALANCED
#define LOCKS_SCAN_BALANCED 1  // tensor scan: deal (problem, group) units to the warps by actual lengths (0: equal warps per problem)
#endif
#ifndef LOCKS_SCAN_HINT_LOAD
#define LOCKS_SCAN_HINT_LOAD 1    // tensor scan: summaries are read with an L2 evict-first policy
#endif
#ifndef LOCKS_SCAN_HINT_STORE
#define LOCKS_SCAN_HINT_STORE 1   // tensor scan: scores are written with an L2 evict-last policy
#endif
#ifndef LOCKS_ATT_HINT_LOAD
#define LOCKS_ATT_HINT_LOAD 1     // sparse attention: K and V tiles are read with an L2 evict-first policy
#endif
#ifndef LOCKS_SCAN_BULK
#define LOCKS_SCAN_BULK 1      // staging of summary blobs in the scan: 1 = cp.async.bulk (TMA) + mbarrier, 0 = 16-byte cp.async
#endif
#define LOCKS_SPIN_LIMIT (1 << 22)  // bounded mbarrier polling (each poll already waits a while) ...
#define LOCKS_WAIT_LIMIT_NS 1000000000ull   // ... and never longer than a second

// One cached CUDA graph of the host-buffer decode step (copies in, step, copies out) for one set of arguments.
struct locks_host_graph {
  const void *q, *kn, *vn;
  void *out, *summ;
  int32_t *ids, *cnt;
  locks_kv kv;
  int batch;
  cudaStream_t st;
  int seen;                 // eager calls made with these arguments
  int launches;
  cudaGraphExec_t exec;     // nullptr until the arguments have been seen twice
};
#define LOCKS_HOST_GRAPHS 8

struct locks_ctx {
  locks_config cfg;
  int G, k, S, Pmax, max_groups;
  int B;                   // tokens per page (cfg.page_size): 16, or 32 / 64 on the plain kernels
  int num_sms;
  int part_slots;          // partial slots per (request, head) the last scan launch may have filled
  int part_balanced;       // the last scan launch wrote per-problem partial counts to part_cnt instead
  int scan_partition;      // LOCKS_PARTITION_*: how the tensor scan deals pages to its warps
  int last_partition;      // partition the last tensor-scan launch used (0: no such launch yet)
  int scorer;              // LOCKS_SCORER_*: what the next scan launch computes per page (diagnostics switch it)
  int32_t *hint_host;      // pinned, device-mapped word: partition the device suggests for the current lengths
  int32_t *hint_dev;       //   (0 none yet, LOCKS_PARTITION_STRIDED, LOCKS_PARTITION_BALANCED)
  int sel_ept;             // pages per thread of a selector CTA (chunk = sel_ept * 512 pages)
  int sel_chunks;          // selector CTAs (chunks) per (request, KV head)
  int sel_kc;              // candidates kept per chunk (k-2)
  // workspace partition (device)
  char *ws;
  size_t ws_bytes;
  int32_t *status;         // [4] sticky status, work counters
  float *shat;             // [max_batch][Hq][Pmax]
  float2 *part;            // [max_batch][Hq][max_groups] partial (max, sum exp) over candidate pages
  int32_t *part_cnt;       // [max_batch][Hkv] partials the scan wrote per head of a problem (balanced partition)
  int32_t *sel_done;       // [max_batch][Hkv] chunk-arrival counters
  float *cand_val;         // [max_batch][Hkv][sel_chunks][sel_kc] chunk lists: 32-bit keys (0 = no entry)
  int32_t *cand_idx;
  float *att_o;            // [rows][d], rows = batch * Hq * splits <= att_rows
  float *att_lse;          // [rows]  (log2 units)
  int32_t *att_done;       // [max_batch][Hkv] split-arrival counters
  int32_t *ids_int;        // [max_batch][Hkv][k]
  int32_t *cnt_int;        // [max_batch][Hkv]
  char *stage_q, *stage_kn, *stage_vn, *stage_out;
  int32_t *seq_eff;        // [2][max_batch] decode step in flight: effective lengths, append positions
  cudaStream_t side;       // build of freshly filled pages runs beside attend
  cudaEvent_t ev_fork, ev_join;
  int last_launches;
  locks_host_graph hg[LOCKS_HOST_GRAPHS];
  int hg_next;
  int att_cluster_max;     // largest thread-block cluster the attention kernel may use (-1: not probed yet)
  // optional per-stage timing of eager decode steps (see locks_profile_begin)
  cudaEvent_t *prof_ev;    // [prof_cap][LOCKS_PROF_MARKS]
  int prof_cap, prof_n;
};
#define LOCKS_PROF_MARKS 4   // step start, after scan, after select, after attend

// The new token of a decode step, handed to the selector's first kernel, which writes it into the cache.
struct locks_append {
  const void *k_new, *v_new;   // [batch][Hkv][d]; k_new == nullptr: nothing to append
  void *k, *v;
  int64_t sb, sh, st;          // cache strides in elements
  const int32_t *block_table;
  const int32_t *seq_eff;      // published by the scan: [batch] lengths, [batch] append positions
  int32_t *seq_commit;         // the caller's sequence lengths
  int num_blocks, esz;
};

// Geometry of a tensor-scan launch: known on the host, used by the launcher and by the partition hint
struct locks_scan_geom {
  int grid, W;               // CTAs, warps
  int wpp, nslots, rounds;   // strided partition: warps per problem, problems in flight, problems per slot
  int cta_reduce;            // all warps of a CTA share one problem for the whole launch
};
locks_scan_geom locks_scan_geometry(const locks_ctx *c, int batch);

// Which partition suits these lengths: iterations of the longest warp, strided = rounds * ceil(max groups / wpp)
// against balanced = ceil(units / warps); the balanced one has to win by more than its set-up costs.
// Called by one warp; lane 0 writes *hint.
__device__ __forceinline__ void locks_update_partition_hint(int32_t *hint, const int32_t *seq_lens, int batch, int Hkv,
                                                            int k, int wpp, int rounds, int W, int lane) {
  int sum = 0, mx = 0;
  for (int b = lane; b < batch; b += 32) {
    const int P = (seq_lens[b] + LOCKS_B - 1) / LOCKS_B;   // (the hint serves the tensor scan: 16-token pages)
    const int ng = P <= k ? 0 : (P - 1 + LOCKS_GROUP - 1) / LOCKS_GROUP;
    sum += ng;
    mx = max(mx, ng);
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  if (lane == 0) {
    const int strided = rounds * ((mx + wpp - 1) / wpp);
    const int even = (int)(((int64_t)sum * Hkv + W - 1) / W);
    *hint = (strided * 16 > even * 17 + 8) ? LOCKS_PARTITION_BALANCED : LOCKS_PARTITION_STRIDED;
  }
}

// launchers (each returns LOCKS_OK or LOCKS_ERR_CUDA and adds to ctx->last_launches)
// seq_inc = 1: lengths are taken one token longer than kv->seq_lens says and published in ctx->seq_eff
int locks_launch_scan(locks_ctx *c, const void *q, const void *summaries, const locks_kv *kv, int batch,
                      float *shat, int seq_inc, cudaStream_t st);
int locks_launch_select(locks_ctx *c, const float *shat, const locks_kv *kv, int batch, int32_t *ids,
                        int32_t *cnt, float *logshare, const locks_append *app, cudaStream_t st);
int locks_launch_attend(locks_ctx *c, const void *q, const locks_kv *kv, int batch, const int32_t *ids,
                        const int32_t *cnt, void *out, float *lse, cudaStream_t st);
int locks_launch_build(locks_ctx *c, const locks_kv *kv, int batch, const int32_t *pb, const int32_t *pe,
                       int just_filled, void *summaries, const void *k_new, const int32_t *append_pos,
                       cudaStream_t st, const void *const *k_layers = nullptr, void *const *summ_layers = nullptr,
                       int num_layers = 1);

// envelope = 0: exact page log-mass; 1: the min/max envelope bound of the page's largest logit
int locks_launch_exact_scan(locks_ctx *c, const void *q, const locks_kv *kv, int batch, float *shat, int envelope,
                            cudaStream_t st);
int locks_launch_quality(locks_ctx *c, const float *mass, const locks_kv *kv, int batch, const int32_t *ids_a,
                         const int32_t *cnt_a, const int32_t *ids_r, const int32_t *cnt_r, const int32_t *marked,
                         int n_marked, float *out, cudaStream_t st);

int locks_launch_head_logz(locks_ctx *c, const locks_kv *kv, int batch, float *logz, cudaStream_t st);
int locks_launch_ext_partials(locks_ctx *c, const float *logz_parts, int nparts, int batch, cudaStream_t st);
int locks_launch_merge_selection(locks_ctx *c, const float *cand_key, const int32_t *cand_page, int nparts, int batch,
                                 int32_t *ids, int32_t *cnt, cudaStream_t st);
int locks_launch_merge_shards(locks_ctx *c, const void *part_out, const float *part_lse, int nparts, int batch, void *out,
                              float *lse, cudaStream_t st);
int locks_launch_fake_quant(locks_ctx *c, const locks_kv *kv, int batch, const int32_t *pb, const int32_t *pe, int bits,
                            cudaStream_t st);

// Launch with programmatic dependent launch allowed: the kernel may be scheduled while its stream
// predecessor is still draining; it must execute pdl_wait() before touching anything the predecessor
// writes (the wait returns once the predecessor grid has completed and its writes are visible).
template <typename... KArgs, typename... Args>
static inline void locks_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, args...);
}

// The same, with the grid's x dimension grouped into thread-block clusters of `cluster_x` CTAs
// (distributed shared memory between the CTAs of a cluster).
template <typename... KArgs, typename... Args>
static inline void locks_launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, int cluster_x,
                                            cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = cluster_x;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  (void)cudaLaunchKernelEx(&cfg, kernel, args...);
}

// A failed launch is reported once: the runtime's sticky-until-read error is cleared, so that the next call
// on this thread is judged on its own launches.
static inline int locks_check_launch(locks_ctx *c) {
  c->last_launches++;
  if (cudaPeekAtLastError() == cudaSuccess) return LOCKS_OK;
  (void)cudaGetLastError();
  return LOCKS_ERR_CUDA;
}

// Function attributes (dynamic shared-memory limit, non-portable cluster size) belong to a device, not to the
// process: true exactly once per (current device, kernel family), so that a process that drives several GPUs
// sets them on each.  Thread-safe.
enum { LOCKS_ATTR_SELECT = 0, LOCKS_ATTR_ATTEND = 1, LOCKS_ATTR_EXACT = 3, LOCKS_ATTR_BUILD = 4 /* + format */, LOCKS_ATTR_SCAN = 8,
       LOCKS_ATTR_BUILD_WIDE = 24 /* + format */ };
bool locks_attrs_needed(int family);

// ---------------------------------------------------------------- I4 blob geometry (d = 128; B = 16 unless given)
// [basis 64 r][coefficients B r][centroid 128][sC B x fp16][sV r x fp16][sMu fp16], padded to 16.
__host__ __device__ constexpr int i4_off_coef(int r) { return 64 * r; }
__host__ __device__ constexpr int i4_off_mu(int r, int B = LOCKS_B) { return 64 * r + B * r; }
__host__ __device__ constexpr int i4_off_sc(int r, int B = LOCKS_B) { return i4_off_mu(r, B) + 128; }
__host__ __device__ constexpr int i4_off_sv(int r, int B = LOCKS_B) { return i4_off_sc(r, B) + 2 * B; }
__host__ __device__ constexpr int i4_off_smu(int r, int B = LOCKS_B) { return i4_off_sv(r, B) + 2 * r; }
__host__ __device__ constexpr int i4_stride(int r, int B = LOCKS_B) { return (i4_off_smu(r, B) + 2 + 15) / 16 * 16; }
__host__ __device__ constexpr int f32_stride(int r, int B = LOCKS_B) { return 4 * (LOCKS_D + r * LOCKS_D + B * r); }
// Row-major formats with an int8 (wide = 1) or bf16 (wide = 2) basis:
// [basis r x d][coefficients B x r][centroid d][sC B x fp16][sV r x fp16 (int8 basis only)][sMu fp16], padded to 16.
__host__ __device__ constexpr int wb_off_coef(int r, int wide) { return wide * LOCKS_D * r; }
__host__ __device__ constexpr int wb_off_mu(int r, int wide, int B = LOCKS_B) { return wide * LOCKS_D * r + B * r; }
__host__ __device__ constexpr int wb_off_sc(int r, int wide, int B = LOCKS_B) { return wb_off_mu(r, wide, B) + LOCKS_D; }
__host__ __device__ constexpr int wb_off_sv(int r, int wide, int B = LOCKS_B) { return wb_off_sc(r, wide, B) + 2 * B; }
__host__ __device__ constexpr int wb_off_smu(int r, int wide, int B = LOCKS_B) { return wb_off_sv(r, wide, B) + (wide == 1 ? 2 * r : 0); }
__host__ __device__ constexpr int wb_stride(int r, int wide, int B = LOCKS_B) { return (wb_off_smu(r, wide, B) + 2 + 15) / 16 * 16; }
__host__ __device__ constexpr int locks_fmt_stride(int fmt, int r, int B = LOCKS_B) {
  return fmt == LOCKS_FMT_I4 ? i4_stride(r, B) : fmt == LOCKS_FMT_F32 ? f32_stride(r, B) : wb_stride(r, fmt == LOCKS_FMT_BF16 ? 2 : 1, B);
}

#ifdef __CUDACC__

__device__ __forceinline__ void set_status(int32_t *status, int code) { atomicCAS(status, 0, code); }

// programmatic dependent launch: wait for the stream predecessor / let the successor be scheduled
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <typename T> __device__ __forceinline__ float ldf(const T *p, int64_t i);
template <> __device__ __forceinline__ float ldf<float>(const float *p, int64_t i) { return p[i]; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p, int64_t i) {
  return __bfloat162float(p[i]);
}
template <typename T> __device__ __forceinline__ void stf(T *p, int64_t i, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, int64_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, int64_t i, float v) {
  p[i] = __float2bfloat16_rn(v);
}

// D (16x8, fp32) += A (16x16, row) * B (16x8, col), bf16 or fp16 operands.
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier + bulk async copy (TMA engine, untiled form) ------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t *bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
// Bounded wait on a phase parity: true when the phase completed, false when the poll limit ran out.
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Waits for the phase `parity` of an mbarrier.  Bounded twice: by a number of polls and by wall time (the
// clock is read only after a poll has failed).  false = the wait ran out; the caller reports LOCKS_ERR_TIMEOUT.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, uint64_t limit_ns = LOCKS_WAIT_LIMIT_NS) {
  uint32_t a = smem_u32(bar);
  uint64_t t0 = 0;
  for (int it = 0; it < LOCKS_SPIN_LIMIT; ++it) {
    uint32_t done;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                 " selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(done)
                 : "r"(a), "r"(parity)
                 : "memory");
    if (done) return true;
    if (it == 0) t0 = global_ns();
    else if (global_ns() - t0 > limit_ns) return false;
  }
  return false;
}
// global -> shared bulk copy; size multiple of 16, both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::
                   "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// L2 eviction policies: a stream that is read once should not push out what the next kernel reads
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(void *dst, const void *src, uint32_t bytes, uint64_t *bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n" ::
                   "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void st_f32_hint(float *dst, float v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;\n" ::"l"(dst), "f"(v), "l"(pol) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}

// ---- Ampere-style 16-byte async copies --------------------------------------------------------
__device__ __forceinline__ void cp_async16(void *dst, const void *src, bool valid) {
  int sz = valid ? 16 : 0;  // src-size 0 zero-fills the destination
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_u32(dst)), "l"(src), "r"(sz)
               : "memory");
}
// With an L2 cache policy.  The policy operand is only ever combined with a full 16-byte copy: the hinted
// form with a source size below the copy size (the zero-fill idiom) raised "illegal instruction" on sm_100a,
// so rows to be zero-filled take the plain form.
__device__ __forceinline__ void cp_async16_hint(void *dst, const void *src, bool valid, uint64_t pol) {
  if (valid)
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(smem_u32(dst)), "l"(src), "l"(pol)
                 : "memory");
  else
    cp_async16(dst, src, false);
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void *p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void *p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

#endif  // __CUDACC__
