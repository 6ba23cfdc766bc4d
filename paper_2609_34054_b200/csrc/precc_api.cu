// C-ABI entry points of libprecc: argument validation, launch configuration, kernel dispatch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "../../include/precc.h"
#include "decode.cuh"
#include "combine.cuh"
#include "gemm_tc.cuh"
#include "proj_small.cuh"
#include "prefill.cuh"
#include "prefill_tc.cuh"

using namespace precc;

struct precc_ctx {
  int device = 0;
  int sm_count = 0;
  int max_smem_optin = 0;
  uint32_t* status = nullptr;          // device status word
  unsigned long long* trace = nullptr; // optional caller-owned trace buffer
  size_t trace_blocks = 0;
  bool force_simple_prefill = false;   // PRECC_PREFILL=simple in the environment
  bool force_tiled_gemm = false;       // PRECC_GEMM=tiled in the environment: never take the few-row kernel
  bool no_gemm_splitk = false;         // PRECC_GEMM_SPLITK=0 in the environment: short turns stay on the one-block-per-tile GEMM
  bool force_ticket_decode = false;    // PRECC_DECODE=ticket in the environment: never use the cluster decode kernel
  bool deep_clusters = true;           // PRECC_DEEP=0 in the environment: never use the one-block-per-SM deep-ring clusters
  bool prefill_forward = false;        // PRECC_PREFILL_ORDER=forward: row tiles in ascending order (default: longest causal reach first)
  bool no_prefill_split = false;       // PRECC_PREFILL_SPLIT=0 in the environment: never split a turn's context over a cluster
  char err[512] = {0};
  CUresult (*encode_tiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                           const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                           CUtensorMapL2promotion, CUtensorMapFloatOOBfill) = nullptr;
};

// Scratch for precc_lr_attend_decode_static: lives in the library image, one copy per GPU that loads it.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[PRECC_STATIC_SCRATCH_BYTES];

namespace {

// Device address of g_static_scratch on each device, looked up on the first static call there.
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {nullptr};

int32_t fail(precc_ctx* ctx, int32_t code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

#define PRECC_CUDA(ctx, expr)                                                                   \
  do {                                                                                          \
    cudaError_t e__ = (expr);                                                                   \
    if (e__ != cudaSuccess) return fail(ctx, PRECC_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

// Dynamic shared-memory limit of a kernel on the context's device: only ever raised (a kernel serves
// several configurations; lowering the limit for a small one would make a later large launch fail), and
// set under a lock so that contexts on several host threads cannot interleave a set and a launch badly.
struct SmemLimit { const void* fn; int dev; int bytes; };
std::mutex g_limits_mu;
SmemLimit g_limits[1024];
int g_n_limits = 0;
template <typename K>
cudaError_t raise_smem_limit(precc_ctx* ctx, K kern, int bytes) {
  const void* fn = reinterpret_cast<const void*>(kern);
  std::lock_guard<std::mutex> lk(g_limits_mu);
  SmemLimit* e = nullptr;
  for (int i = 0; i < g_n_limits; ++i)
    if (g_limits[i].fn == fn && g_limits[i].dev == ctx->device) { e = &g_limits[i]; break; }
  if (e && bytes <= e->bytes) return cudaSuccess;
  const cudaError_t rc = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (rc != cudaSuccess) return rc;
  if (!e && g_n_limits < 1024) { e = &g_limits[g_n_limits++]; e->fn = fn; e->dev = ctx->device; e->bytes = 0; }
  if (e) e->bytes = bytes;
  return cudaSuccess;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool rank_ok(int r) { return r == 8 || r == 16 || r == 32 || r == 64; }

int32_t check_desc(precc_ctx* ctx, const precc_layer_desc* d) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!d) return fail(ctx, PRECC_ERR_INVALID_ARG, "layer descriptor is null");
  if (d->d_model <= 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->n_agents <= 0 || d->rank_k < 0 || d->rank_v < 0)
    return fail(ctx, PRECC_ERR_INVALID_ARG, "non-positive size in layer descriptor");
  if (d->head_dim != 64 && d->head_dim != 128) return fail(ctx, PRECC_ERR_UNSUPPORTED, "head_dim %d not in {64,128}", d->head_dim);
  if (d->n_q_heads % d->n_kv_heads) return fail(ctx, PRECC_ERR_UNSUPPORTED, "n_q_heads %% n_kv_heads != 0");
  if (d->n_q_heads / d->n_kv_heads > 8) return fail(ctx, PRECC_ERR_UNSUPPORTED, "group size %d > 8", d->n_q_heads / d->n_kv_heads);
  if (d->d_model % 64) return fail(ctx, PRECC_ERR_UNSUPPORTED, "d_model %d not a multiple of 64", d->d_model);
  if (d->n_agents > 64) return fail(ctx, PRECC_ERR_UNSUPPORTED, "n_agents %d > 64", d->n_agents);
  const int rk = d->rank_k, rv = d->rank_v;
  const bool combo = (rk == 0 && rv == 0) || (rk == 0 && rank_ok(rv)) || (rk == rv && rank_ok(rv));
  if (!combo) return fail(ctx, PRECC_ERR_UNSUPPORTED, "ranks (%d,%d) not in {(0,0),(0,r),(r,r)}, r in {8,16,32,64}", rk, rv);
  return PRECC_OK;
}

int32_t check_cache(precc_ctx* ctx, const precc_layer_desc* d, const precc_cache* c, bool need_base, bool need_lr) {
  if (!c) return fail(ctx, PRECC_ERR_INVALID_ARG, "cache is null");
  if (c->n_blocks <= 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "cache.n_blocks must be positive");
  if (c->n_blocks > (int64_t)1 << 26) return fail(ctx, PRECC_ERR_UNSUPPORTED, "cache.n_blocks too large");
  if (need_base && (!c->k_base || !c->v_base)) return fail(ctx, PRECC_ERR_INVALID_ARG, "base cache pointer is null");
  if (need_lr && ((d->rank_k > 0 && !c->lr_k) || (d->rank_v > 0 && !c->lr_v))) return fail(ctx, PRECC_ERR_INVALID_ARG, "LR cache pointer is null");
  if (!aligned16(c->k_base) || !aligned16(c->v_base) || !aligned16(c->lr_k) || !aligned16(c->lr_v))
    return fail(ctx, PRECC_ERR_MISALIGNED, "cache pointer not 16-byte aligned");
  return PRECC_OK;
}

float softmax_scale_log2(const precc_layer_desc* d) {
  const float sc = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / std::sqrt((float)d->head_dim);
  return sc * 1.4426950408889634f;
}

// ------------------------------------------------------------------------------------------ pack
// dst is k-blocked: element (row, i) lives at ((i / 64) * dst_rows + row) * 64 + i % 64, so the 64-deep k
// step of any range of rows is one contiguous run in memory (what a TMA box of the GEMMs fetches).
__global__ void pack_kmajor_kernel(const __nv_bfloat16* __restrict__ src, int d, int n, __nv_bfloat16* __restrict__ dst, int dst_rows,
                                   int row0) {
  __shared__ __nv_bfloat16 tile[32][33];
  const int c0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int i = i0 + r, c = c0 + threadIdx.x;
    tile[r][threadIdx.x] = (i < d && c < n) ? src[(size_t)i * n + c] : __float2bfloat16(0.f);
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int c = c0 + r, i = i0 + threadIdx.x;
    if (c < n && i < d) dst[((size_t)(i / GEMM_BK) * dst_rows + row0 + c) * GEMM_BK + i % GEMM_BK] = tile[threadIdx.x][r];
  }
}

// ------------------------------------------------------------------------------------ GEMM launch
int32_t make_map(precc_ctx* ctx, CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)GEMM_BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, PRECC_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return PRECC_OK;
}

// Tensor map over a k-blocked packed weight matrix [K/64][rows][64]: box = `box_rows` rows of one k block.
int32_t make_map_w(precc_ctx* ctx, CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
  const cuuint64_t dims[3] = {(cuuint64_t)GEMM_BK, (cuuint64_t)rows, (cuuint64_t)(K / GEMM_BK)};
  const cuuint64_t strides[2] = {(cuuint64_t)GEMM_BK * 2, (cuuint64_t)rows * GEMM_BK * 2};
  const cuuint32_t box[3] = {(cuuint32_t)GEMM_BK, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, PRECC_ERR_CUDA, "cuTensorMapEncodeTiled (packed weights) failed (%d)", (int)r);
  return PRECC_OK;
}

// 2-D bf16 tensor map: `rows` x `cols` (cols contiguous), box `box_rows` x `box_cols`, swizzle = box row bytes.
int32_t make_map2(precc_ctx* ctx, CUtensorMap* map, const void* base, long long rows, int cols, int box_rows, int box_cols) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const int bytes = box_cols * 2;
  const CUtensorMapSwizzle sw = bytes >= 128 ? CU_TENSOR_MAP_SWIZZLE_128B : bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, PRECC_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return PRECC_OK;
}

// Column tile width.  A block's time per 64-deep k-block hardly depends on the width below 256 columns (the
// thread that issues the MMAs needs about a hundred cycles per instruction, four per k-block: measured 0.52 us
// per k-block at 256 columns, 0.45 at 128, 0.42 at 64 and still 0.40 at 16), so a launch costs about
// rounds x that, rounds = ceil(tiles / SMs): the widest tile that does not add a round wins
// (2048 rows x 2304 columns: 144 tiles of 256 in one round, 35 us, against 288 tiles of 128 in two, 55 us).
int pick_bn(int n_out, int m_tiles, int sm_count) {
  if (n_out <= 256) return (n_out + 15) / 16 * 16;
  const int cands[3] = {256, 128, 64};
  const double per_kblock[3] = {0.52, 0.45, 0.42};
  int best = 256;
  double best_cost = 1e30;
  for (int i = 0; i < 3; ++i) {
    const long long tiles = (long long)m_tiles * ((n_out + cands[i] - 1) / cands[i]);
    const double cost = (double)((tiles + sm_count - 1) / sm_count) * per_kblock[i];
    if (cost < best_cost - 1e-9) { best_cost = cost; best = cands[i]; }
  }
  return best;
}

// Few rows (decode steps): the weight-streaming split-K kernel.  The K split depends on K alone, so a
// column's summation order - and with it every output bit - is the same whichever entry point (LR only,
// base only, fused) produced it.
int32_t launch_small(precc_ctx* ctx, const void* X, int M, int K, const void* Wt, int n_out, GemmParams gp, cudaStream_t stream) {
  int cs = 8;
  while (cs > 1 && (K / cs < 512 || K % (PS_BK * cs) != 0)) cs >>= 1;
  const int k_slice = K / cs;
  const int steps = k_slice / PS_BK;
  int mt = M <= 16 ? 1 : (M <= 32 ? 2 : 4);
  if (gp.rope && ps_cols(mt) % gp.hd != 0) mt = 2;     // a head's two halves must sit in one block tile (128 columns)
  const int smem = ps_smem_bytes(mt);
  if (steps < 1 || smem > ctx->max_smem_optin) return -1;                // caller falls back to the tiled kernel
  gp.M = M; gp.N_out = n_out; gp.K = K; gp.status = ctx->status;
  const int cols = ps_cols(mt);
  CUtensorMap map_x, map_w;
  int32_t rc = make_map(ctx, &map_x, X, M, K, mt * 16);
  if (rc) return rc;
  rc = make_map_w(ctx, &map_w, Wt, n_out, K, cols);
  if (rc) return rc;
  const int groups = (n_out + cols - 1) / cols;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(groups * cs);
  cfg.blockDim = dim3(PS_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cs; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  auto go = [&](auto kern) -> int32_t {
    PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, smem));
    PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, kern, map_x, map_w, gp, k_slice));
    return PRECC_OK;
  };
  if (mt == 1) return go(proj_small_kernel<1>);
  if (mt == 2) return go(proj_small_kernel<2>);
  return go(proj_small_kernel<4>);
}

int32_t launch_gemm(precc_ctx* ctx, const void* X, int M, int K, const void* Wt, int n_out, GemmParams gp, cudaStream_t stream) {
  // Up to 40 rows the weight-streaming few-row kernel is the fastest (fused C3 projection: 8.7 us at 16 rows, 11.6 at
  // 32); from there to 512 rows the split-K kernel (13..24 us; the few-row kernel needs 16.5 us at 48 rows and 18.4 at
  // 64, the one-block-per-tile GEMM 27 us throughout); the few-row kernel still takes 41..64 rows when the split does
  // not apply (rotary epilogue, short K).
  if (M <= 40 && !ctx->force_tiled_gemm) {
    const int32_t rc = launch_small(ctx, X, M, K, Wt, n_out, gp, stream);
    if (rc >= 0) return rc;
  }
  const int m_tiles = (M + GEMM_BM - 1) / GEMM_BM;
  // A few row tiles (the tokens of a short turn): the K extent of every tile is split over a cluster.  The split
  // depends on M and K alone, so a column's summation order is the same whichever entry point produced it.
  if (m_tiles <= 4 && !gp.rope && !ctx->no_gemm_splitk) {
    const int nkb = K / GEMM_BK;
    // planned for the width of the FUSED projection of this layer, whatever this call projects, so that the base-only,
    // LR-only and fused calls of one M take the same decision (and with it the same summation order)
    const int n_fused = 2 * gp.n_kv * gp.hd + gp.n_agents * (gp.rank_k + gp.rank_v);
    // 256-column tiles, one block per SM (a kernel that allocates tensor memory is given one block per SM)
    const int bn = n_out >= 256 ? 256 : (n_out + 15) / 16 * 16;
    const int stage_bytes = GEMM_A_BYTES + 256 * GEMM_BK * 2;
    const int ring_max = 3 * stage_bytes;
    const long long clusters = (long long)m_tiles * ((n_fused + 255) / 256);
    // the finest split whose clusters are all resident at once (a second wave would cost more than the split gains);
    // cluster sizes need not be powers of two: 18 clusters fit as 6-block clusters, 36 as 3-block clusters
    int ks = GEMM_MAX_KS, smem_plan = 0;
    for (; ks > 2; --ks) {                                       // a two-way split does not pay for its merge
      if (nkb / ks < 2) continue;
      const int cw = ((256 + ks - 1) / ks + 7) / 8 * 8;          // planned for the widest tile, whatever this call's width
      const int dump = ks * GEMM_BM * (cw + 4) * 4;
      smem_plan = (((ring_max > dump ? ring_max : dump) + 1023) & ~1023) + (2 * 3 + 4) * 8;
      if (smem_plan > ctx->max_smem_optin) continue;
      static int max_clusters_dev[kMaxDevices][GEMM_MAX_KS + 1] = {{0}};   // 0 = unknown, else max active clusters + 1
      int& cached = max_clusters_dev[ctx->device % kMaxDevices][ks];
      if (cached == 0) {
        int n = 0;
        if (raise_smem_limit(ctx, proj_gemm_splitk_kernel, smem_plan) == cudaSuccess) {
          cudaLaunchConfig_t qc = {};
          qc.gridDim = dim3(ks, ctx->sm_count, 1); qc.blockDim = dim3(GEMM_THREADS); qc.dynamicSmemBytes = smem_plan;
          cudaLaunchAttribute qa[1];
          qa[0].id = cudaLaunchAttributeClusterDimension;
          qa[0].val.clusterDim.x = ks; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
          qc.attrs = qa; qc.numAttrs = 1;
          if (cudaOccupancyMaxActiveClusters(&n, proj_gemm_splitk_kernel, &qc) != cudaSuccess) { cudaGetLastError(); n = 0; }
        } else {
          cudaGetLastError();
        }
        cached = n + 1;
      }
      if (cached - 1 >= clusters) break;
    }
    if (ks > 2) {
      const int n_tiles = (n_out + bn - 1) / bn;
      int stages = 3;
      if (stages > nkb / ks) stages = nkb / ks;
      int tmem_cols = 32;
      while (tmem_cols < bn) tmem_cols <<= 1;
      CUtensorMap map_x, map_w;
      int32_t rc = make_map(ctx, &map_x, X, M, K, GEMM_BM);
      if (rc) return rc;
      rc = make_map_w(ctx, &map_w, Wt, n_out, K, bn);
      if (rc) return rc;
      gp.M = M; gp.N_out = n_out; gp.K = K; gp.BN = bn; gp.stages = stages; gp.tmem_cols = tmem_cols;
      gp.spread_rows = 0;
      gp.status = ctx->status;
      PRECC_CUDA(ctx, raise_smem_limit(ctx, proj_gemm_splitk_kernel, smem_plan));
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(ks, n_tiles, m_tiles);
      cfg.blockDim = dim3(GEMM_THREADS);
      cfg.dynamicSmemBytes = smem_plan;
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = ks; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, proj_gemm_splitk_kernel, map_x, map_w, gp));
      return PRECC_OK;
    }
  }
  if (M <= PS_MAX_M && !ctx->force_tiled_gemm) {
    const int32_t rc = launch_small(ctx, X, M, K, Wt, n_out, gp, stream);
    if (rc >= 0) return rc;
  }
  int bn = pick_bn(n_out, m_tiles, ctx->sm_count);
  if (gp.rope && bn % gp.hd != 0) bn = gp.hd;        // a head's two halves must sit in one tile
  const int n_tiles = (n_out + bn - 1) / bn;
  const int stage_bytes = GEMM_A_BYTES + bn * GEMM_BK * 2;
  int stages = (ctx->max_smem_optin - 4096) / stage_bytes;
  if (stages > 8) stages = 8;
  if (stages > K / GEMM_BK) stages = K / GEMM_BK;
  if (stages < 1) return fail(ctx, PRECC_ERR_CUDA, "not enough shared memory for one GEMM stage");
  int tmem_cols = 32;
  while (tmem_cols < 2 * bn) tmem_cols <<= 1;      // two accumulator buffers
  const size_t smem = (size_t)stages * stage_bytes + (2 * stages + 6) * 8 + 1024;
  CUtensorMap map_x, map_w;
  int32_t rc = make_map(ctx, &map_x, X, M, K, GEMM_BM);
  if (rc) return rc;
  rc = make_map_w(ctx, &map_w, Wt, n_out, K, bn);
  if (rc) return rc;
  gp.M = M; gp.N_out = n_out; gp.K = K; gp.BN = bn; gp.stages = stages; gp.tmem_cols = tmem_cols;
  gp.spread_rows = 1;
  gp.status = ctx->status;
  PRECC_CUDA(ctx, raise_smem_limit(ctx, proj_gemm_kernel, (int)smem));
  const int total_tiles = m_tiles * n_tiles;
  proj_gemm_kernel<<<dim3(total_tiles < ctx->sm_count ? total_tiles : ctx->sm_count), GEMM_THREADS, smem, stream>>>(map_x, map_w, gp);
  PRECC_CUDA(ctx, cudaGetLastError());
  return PRECC_OK;
}

// ---------------------------------------------------------------------------- attention dispatch
template <template <int, int, int> class F, typename... Args>
int32_t dispatch_shape(precc_ctx* ctx, int hd, int rk, int rv, Args&&... args) {
#define PRECC_CASE(HD, RK, RV) \
  if (hd == HD && rk == RK && rv == RV) return F<HD, RK, RV>::run(ctx, args...);
#define PRECC_RANKS(HD)                                                                              \
  PRECC_CASE(HD, 0, 0) PRECC_CASE(HD, 0, 8) PRECC_CASE(HD, 0, 16) PRECC_CASE(HD, 0, 32) PRECC_CASE(HD, 0, 64) \
  PRECC_CASE(HD, 8, 8) PRECC_CASE(HD, 16, 16) PRECC_CASE(HD, 32, 32) PRECC_CASE(HD, 64, 64)
  PRECC_RANKS(64)
  PRECC_RANKS(128)
#undef PRECC_RANKS
#undef PRECC_CASE
  return fail(ctx, PRECC_ERR_UNSUPPORTED, "no kernel for head_dim %d ranks (%d,%d)", hd, rk, rv);
}

// Split schedule of decode.  cluster > 0: the cluster kernel with that many blocks per (request, kv head);
// otherwise the ticket kernel with up to max_splits blocks per (request, kv head).
struct DecodePlan { int cluster, warps, chunk_tiles, max_splits, stages, smem, deep; };

// `extra`: bytes of shared memory appended after the usual layout (the rotary variant's B_k slice).
template <int HD, int RK, int RV>
DecodePlan plan_ticket(int sm_count, int max_smem, int B, int n_kv, int max_ctx, int extra = 0) {
  using C = DecodeCfg<HD, RK, RV>;
  DecodePlan pl{};
  // ring depth: as deep as possible (<= 4) while two blocks still fit on an SM
  int stages = 4;
  while (stages > 2 && 2 * (C::ticket_smem(stages) + extra + 1024) > max_smem) --stages;
  pl.stages = stages;
  pl.smem = C::ticket_smem(stages) + extra;
  const int per_sm = (2 * (pl.smem + 1024) <= max_smem) ? 2 : 1;
  const long long slots = (long long)sm_count * per_sm;
  const int max_tiles = (max_ctx + PAGE - 1) / PAGE;
  const long long units = (long long)B * n_kv;
  // blocks per (request, kv head): fill the machine once; with plenty of work use 4 waves of
  // blocks so that requests of different length balance out
  long long want = slots / units;                       // rounded down: one full wave, never a wave and a bit
  if (want < 1) want = 1;
  const long long total_tiles = units * max_tiles;
  if (total_tiles >= slots * 4 * 64) want = (4 * slots + units - 1) / units;
  int chunk = (int)((max_tiles + want - 1) / want);
  if (chunk < DEC_WARPS) chunk = DEC_WARPS;
  if ((max_tiles + chunk - 1) / chunk > DEC_MAX_SPLITS) chunk = (max_tiles + DEC_MAX_SPLITS - 1) / DEC_MAX_SPLITS;
  pl.chunk_tiles = chunk;
  pl.max_splits = (max_tiles + chunk - 1) / chunk;
  return pl;
}

// The cluster kernel serves the latency-bound regime: few (request, kv head) units, each worth
// splitting, the whole grid co-resident in one wave.  Returns cluster = 0 when it does not apply.
template <int HD, int RK, int RV>
DecodePlan plan_cluster(int sm_count, int max_smem, int B, int n_kv, int max_ctx, int extra = 0, bool deep_ok = true) {
  using C = DecodeCfg<HD, RK, RV>;
  DecodePlan pl{};
  const int max_tiles = (max_ctx + PAGE - 1) / PAGE;
  const long long units = (long long)B * n_kv;
  if (units * 2 > sm_count || max_tiles <= 16) return pl;  // too many units, or nothing worth splitting
  // two blocks per SM must fit (a 16-block cluster needs 16 free slots inside one GPC, and not every
  // GPC has 16 SMs): 8 warps with a 2-deep ring if that fits, else 4 warps with the deepest ring that does
  const int budget = max_smem / 2 - 1024 - extra;
  int warps = 8, stages = 2;
  if (C::cluster_smem(8, 2) > budget) {
    warps = 4; stages = 4;
    while (stages > 2 && C::cluster_smem(4, stages) > budget) --stages;
    if (C::cluster_smem(4, stages) > budget) return pl;
  }
  // as many blocks per unit as keep the whole grid in one wave (any size up to 16, not only powers of two:
  // 3 requests x 8 heads take 6 blocks each = 144 blocks, where 4 would leave a third of the SMs idle)
  int cs = DEC_MAX_CLUSTER;
  if ((long long)cs * units > sm_count) cs = (int)(sm_count / units);
  if (cs * warps > max_tiles) cs = max_tiles / warps;
  if (cs < 2) return pl;
  // Wide clusters (very few units) with more than a few pages per warp: one block per SM with the whole
  // shared memory as page rings, i.e. two to three times the bytes in flight per SM and fewer dependent DRAM
  // round trips per warp; the run-time occupancy check then shrinks the cluster until all clusters are
  // resident (a 16-block cluster at one block per SM does not fit every GPC).  Measured against the
  // two-blocks-per-SM layout: 8192 tokens x 8 units 9.3 -> 9.0 us, 32768 tokens 31 -> 27 us, 65536 tokens
  // 53 -> 46 us.  With the deep rings switched off, bandwidth-bound sizes go to the ticket kernel instead.
  // Narrow clusters over a lot of data (e.g. 8 requests x 8 kv heads x 32768 tokens: clusters of 2): the work is
  // bandwidth-bound and the ticket kernel, which spreads it over every SM, is faster (rotary keys: 252 against 350 us).
  if (units * max_tiles > 32768 && cs <= 4) return pl;
  // Wide pages (head_dim 128 with rank 32 or 64) leave the two-blocks-per-SM layout only 4 warps with 2-page
  // rings; narrow clusters of such blocks lose to the ticket kernel's larger grid from a few thousand pages on
  // (rank 32, 8192 tokens, 4..8 requests: 35..58 us against 33..51 us; ranks 8 and 16 keep three-page rings and win).
  if (warps == 4 && stages == 2 && cs <= 4 && units * max_tiles >= 6000) return pl;
  if (units * max_tiles > (deep_ok ? 2048 : 32768) && cs > 4) {
    if (!deep_ok) return pl;
    const int big = max_smem - 2048 - extra;
    warps = 8; stages = 4;
    while (stages > 2 && C::cluster_smem(8, stages) > big) --stages;
    if (C::cluster_smem(8, stages) > big) {
      warps = 4; stages = 4;
      while (stages > 2 && C::cluster_smem(4, stages) > big) --stages;
      if (C::cluster_smem(4, stages) > big) return pl;
    }
    pl.deep = 1;
  }
  pl.cluster = cs;
  pl.warps = warps;
  pl.stages = stages;
  pl.smem = C::cluster_smem(warps, stages) + extra;
  pl.chunk_tiles = (max_tiles + cs - 1) / cs;
  pl.max_splits = cs;
  return pl;
}

struct DecodeArgs {
  const precc_layer_desc* d; const void* q; int B; const int32_t* agent_id; const int32_t* ctx_len;
  const int32_t* block_table; int table_stride; const int32_t* first_block; int max_ctx;
  const void* B_k; const void* B_v; const precc_cache* cache; void* out; void* ws; size_t ws_bytes; cudaStream_t stream;
  const float* rope = nullptr; int max_pos = 0;      // rotary variant when rope != null
  float* raw = nullptr;                              // partial-output mode: records instead of `out`
};

template <int HD, int RK, int RV, bool ROPE = false>
struct DecodeRunT {
  // (the rotary variant never needs more than the plain one: its larger blocks only lower the split count)
  // exact need of one call
  static size_t ws_need(int B, int n_kv, int max_splits) {
    const size_t tickets = ((size_t)B * n_kv * 4 + 255) / 256 * 256;
    return tickets + (size_t)B * n_kv * max_splits * DecodeCfg<HD, RK, RV>::PART_STRIDE * 4;
  }
  // Upper bound over EVERY call with at most B requests of at most max_ctx tokens (a smaller batch gets more
  // splits per request, so the need is not monotone in B).  Mirrors plan_ticket: splits <= blocks wanted per
  // unit, splits <= pages / DEC_WARPS, and the four-wave mode can only switch on as the context grows.
  static size_t ws_bytes(int sm_count, int max_smem, int B, int n_kv, int max_ctx) {
    using C = DecodeCfg<HD, RK, RV>;
    int stages = 4;
    while (stages > 2 && 2 * (C::ticket_smem(stages) + 1024) > max_smem) --stages;
    const long long slots = (long long)sm_count * ((2 * (C::ticket_smem(stages) + 1024) <= max_smem) ? 2 : 1);
    const long long max_tiles = (max_ctx + PAGE - 1) / PAGE;
    size_t best = 0;
    for (int b = 1; b <= B; ++b) {
      const long long units = (long long)b * n_kv;
      long long want = slots / units;
      if (want < 1) want = 1;
      if (units * max_tiles >= slots * 4 * 64) want = (4 * slots + units - 1) / units;
      long long bound = (max_tiles + DEC_WARPS - 1) / DEC_WARPS;
      if (bound > want) bound = want;
      if (bound > DEC_MAX_SPLITS) bound = DEC_MAX_SPLITS;
      if (bound < 1) bound = 1;
      const size_t need = ws_need(b, n_kv, (int)bound);
      if (need > best) best = need;
    }
    return best;
  }
  // Can `need` clusters of `cs` blocks be resident at once?  Asked once per (shape, warps, cluster size).
  // The cluster kernel's shared-memory limit is only ever raised: the two ring layouts of one shape (two blocks
  // per SM / one block per SM) need different amounts, and lowering the attribute for the smaller one would
  // make a later launch of the larger one fail.
  // (Function attributes and occupancy answers belong to a device: the caches are indexed by its ordinal.)
  using ClusterKernel = void (*)(const DecodeParams);
  // two blocks per SM (8 warps, head_dim 64) unless the plan uses the one-block-per-SM ring layout
  template <int NW>
  static ClusterKernel cluster_kernel(bool deep) {
    if constexpr (NW == 8 && HD == 64) {
      if (!deep) return lr_attend_decode_cluster_kernel<HD, RK, RV, 8, ROPE, 2>;
    }
    return lr_attend_decode_cluster_kernel<HD, RK, RV, NW, ROPE, 1>;
  }
  template <int NW>
  static cudaError_t ensure_cluster_smem(precc_ctx* ctx, int bytes, bool deep) {
    static bool nonportable_dev[kMaxDevices][2] = {{false}};
    ClusterKernel kern = cluster_kernel<NW>(deep);
    cudaError_t e = raise_smem_limit(ctx, kern, bytes);
    bool& np = nonportable_dev[ctx->device % kMaxDevices][deep ? 1 : 0];
    if (e == cudaSuccess && !np) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e == cudaSuccess) np = true;
    }
    return e;
  }
  template <int NW>
  static bool cluster_fits(precc_ctx* ctx, const DecodePlan& pl, int need) {
    static int cache2[kMaxDevices][2][DEC_MAX_CLUSTER + 1] = {{{0}}};  // 0 = unknown, else max active clusters + 1
    int* cached = cache2[ctx->device % kMaxDevices][pl.deep ? 1 : 0];
    if (cached[pl.cluster] == 0) {
      ClusterKernel kern = cluster_kernel<NW>(pl.deep != 0);
      int n = 0;
      if (ensure_cluster_smem<NW>(ctx, pl.smem, pl.deep != 0) != cudaSuccess) {
        cudaGetLastError();
        cached[pl.cluster] = 1;
        return false;
      }
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(pl.cluster, ctx->sm_count / pl.cluster, 1);
      cfg.blockDim = dim3(NW * 32);
      cfg.dynamicSmemBytes = pl.smem;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = pl.cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
      cached[pl.cluster] = n + 1;
    }
    return cached[pl.cluster] - 1 >= need;
  }
  static int32_t run(precc_ctx* ctx, const DecodeArgs& a) {
    const precc_layer_desc* d = a.d;
    constexpr int extra = ROPE ? DecodeCfg<HD, RK, RV>::BK_BYTES + 128 : 0;
    // The rotary kernel at head_dim 128 is issue-bound (255 registers, 8 warps per SM at most): it gains more from
    // the 128 blocks of the two-blocks-per-SM layout than from deeper rings on 80 SMs (131072 tokens: 141 against 238 us).
    const bool deep_ok = ctx->deep_clusters && !(ROPE && HD == 128);
    DecodePlan pl = plan_cluster<HD, RK, RV>(ctx->sm_count, ctx->max_smem_optin, a.B, d->n_kv_heads, a.max_ctx, extra, deep_ok);
    if (ctx->force_ticket_decode) pl.cluster = 0;
    auto fits = [&](const DecodePlan& q) { return q.warps == 8 ? cluster_fits<8>(ctx, q, a.B * d->n_kv_heads) : cluster_fits<4>(ctx, q, a.B * d->n_kv_heads); };
    if (pl.cluster && pl.deep) {
      const int max_tiles = (a.max_ctx + PAGE - 1) / PAGE;
      while (pl.cluster > 4 && !fits(pl)) { --pl.cluster; pl.chunk_tiles = (max_tiles + pl.cluster - 1) / pl.cluster; pl.max_splits = pl.cluster; }
      if (pl.cluster <= 4) pl.cluster = 0;
    } else if (pl.cluster && !fits(pl)) {
      pl.cluster = 0;
    }
    if (!pl.cluster) {
      pl = plan_ticket<HD, RK, RV>(ctx->sm_count, ctx->max_smem_optin, a.B, d->n_kv_heads, a.max_ctx, extra);
      const size_t need = ws_need(a.B, d->n_kv_heads, pl.max_splits);
      if (!a.ws || a.ws_bytes < need) return fail(ctx, PRECC_ERR_WORKSPACE, "decode workspace: need %zu bytes, got %zu", need, a.ws_bytes);
    }
    DecodeParams p;
    p.q = (const __nv_bfloat16*)a.q; p.out = (__nv_bfloat16*)a.out;
    p.agent_id = a.agent_id; p.ctx_len = a.ctx_len; p.block_table = a.block_table; p.first_block = a.first_block;
    p.k_base = (const __nv_bfloat16*)a.cache->k_base; p.v_base = (const __nv_bfloat16*)a.cache->v_base;
    p.lr_k = (const __nv_bfloat16*)a.cache->lr_k; p.lr_v = (const __nv_bfloat16*)a.cache->lr_v;
    p.B_k = (const __nv_bfloat16*)a.B_k; p.B_v = (const __nv_bfloat16*)a.B_v;
    const size_t tickets = ((size_t)a.B * d->n_kv_heads * 4 + 255) / 256 * 256;
    p.tickets = (int32_t*)a.ws;
    p.part = a.ws ? (float*)((char*)a.ws + tickets) : nullptr;
    p.raw = a.raw;
    p.status = ctx->status;
    p.trace = (ctx->trace && (size_t)pl.max_splits * d->n_kv_heads * a.B <= ctx->trace_blocks) ? ctx->trace : nullptr;
    p.n_blocks = a.cache->n_blocks; p.table_stride = a.table_stride;
    p.n_q = d->n_q_heads; p.n_kv = d->n_kv_heads; p.group = d->n_q_heads / d->n_kv_heads; p.n_agents = d->n_agents;
    p.chunk_tiles = pl.chunk_tiles; p.max_splits = pl.max_splits; p.stages = pl.stages;
    p.scale_log2 = softmax_scale_log2(d); p.s_k = d->lora_scale_k; p.s_v = d->lora_scale_v;
    p.rope = reinterpret_cast<const float4*>(a.rope); p.max_pos = a.max_pos;
    p.bk_off = ROPE ? ((pl.smem - extra + 127) / 128) * 128 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.max_splits, d->n_kv_heads, a.B);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (pl.cluster) {
      cfg.blockDim = dim3(pl.warps * 32);
      attr[1].id = cudaLaunchAttributeClusterDimension;
      attr[1].val.clusterDim.x = pl.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
      cfg.numAttrs = 2;
      if (pl.warps == 8) {
        PRECC_CUDA(ctx, ensure_cluster_smem<8>(ctx, pl.smem, pl.deep != 0));
        PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, cluster_kernel<8>(pl.deep != 0), p));
      } else {
        PRECC_CUDA(ctx, ensure_cluster_smem<4>(ctx, pl.smem, pl.deep != 0));
        PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, cluster_kernel<4>(pl.deep != 0), p));
      }
    } else {
      auto kern = lr_attend_decode_kernel<HD, RK, RV, ROPE>;
      cfg.blockDim = dim3(DEC_WARPS * 32);
      PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, pl.smem));
      PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, kern, p));
    }
    return PRECC_OK;
  }
};

template <int HD, int RK, int RV>
struct DecodeRun : DecodeRunT<HD, RK, RV, false> {};
// Rotary keys: without a key-side adapter (or for the adapter-free view) the rotated base cache is all
// there is, and the position-free kernel is already exact.
template <int HD, int RK, int RV>
struct DecodeRunRope {
  static int32_t run(precc_ctx* ctx, const DecodeArgs& a) {
    if constexpr (RK > 0) return DecodeRunT<HD, RK, RV, true>::run(ctx, a);
    else return DecodeRunT<HD, RK, RV, false>::run(ctx, a);
  }
};

// 4-D map over a base cache [n_blocks][n_kv][16][hd]: box = 64 columns x 16 rows x 1 head x `box_blocks` blocks.
int32_t make_map_cache4(precc_ctx* ctx, CUtensorMap* map, const void* base, long long n_blocks, int n_kv, int hd, int box_blocks) {
  const cuuint64_t dims[4] = {(cuuint64_t)hd, (cuuint64_t)PAGE, (cuuint64_t)n_kv, (cuuint64_t)n_blocks};
  const cuuint64_t strides[3] = {(cuuint64_t)hd * 2, (cuuint64_t)PAGE * hd * 2, (cuuint64_t)n_kv * PAGE * hd * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)PAGE, 1, (cuuint32_t)box_blocks};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, PRECC_ERR_CUDA, "cuTensorMapEncodeTiled (4-D cache) failed (%d)", (int)r);
  return PRECC_OK;
}

struct PrefillArgs {
  const precc_layer_desc* d; const void* q; int S; int agent; int T; const int32_t* block_table; int first_block;
  const void* B_k; const void* B_v; const precc_cache* cache; void* out; cudaStream_t stream;
  const float* rope = nullptr; int max_pos = 0;      // rotary variant when rope != null
};

template <int HD, int RK, int RV>
struct PrefillRun {
  // tensor-core kernel (tcgen05 + TMEM + TMA) for the shapes it supports
  static int32_t run_tc(precc_ctx* ctx, const PrefillArgs& a) {
    using C = PrefillTcCfg<HD, RK, RV>;
    const precc_layer_desc* d = a.d;
    const int G = d->n_q_heads / d->n_kv_heads;
    // as deep as shared memory allows, keys first (they are needed one step earlier)
    // (head_dim 128 with rank 64 has room for a single value stage: 48 KB per stage of either kind)
    int ks = 2, vs = 1;
    if (C::smem_bytes(ks, vs) > ctx->max_smem_optin) return run_simple<false>(ctx, a);
    while (ks + vs < 8) {
      if (ks <= vs && C::smem_bytes(ks + 1, vs) <= ctx->max_smem_optin) ++ks;
      else if (C::smem_bytes(ks, vs + 1) <= ctx->max_smem_optin) ++vs;
      else break;
    }
    const int smem = C::smem_bytes(ks, vs);
    const size_t kvw = (size_t)d->n_kv_heads * HD;
    const long long kv_rows = (long long)a.cache->n_blocks * d->n_kv_heads * PAGE;
    const long long lr_rows = (long long)a.cache->n_blocks * PAGE;
    CUtensorMap mk, mv, mlk, mlv;
    // without a block table the pages of a 128-token stage are consecutive: whole-stage boxes (one TMA
    // instruction per 64-column slab instead of one per page)
    const bool contig = a.block_table == nullptr;
    const int box_rows = contig ? PTC_TOK : PAGE;
    int32_t rc = contig ? make_map_cache4(ctx, &mk, a.cache->k_base, a.cache->n_blocks, d->n_kv_heads, HD, PTC_TOK / PAGE)
                        : make_map2(ctx, &mk, a.cache->k_base, kv_rows, HD, PAGE, 64);
    if (rc) return rc;
    rc = contig ? make_map_cache4(ctx, &mv, a.cache->v_base, a.cache->n_blocks, d->n_kv_heads, HD, PTC_TOK / PAGE)
                : make_map2(ctx, &mv, a.cache->v_base, kv_rows, HD, PAGE, 64);
    if (rc) return rc;
    mlk = mk; mlv = mv;     // placeholders when a rank is zero (never dereferenced)
    if (RK) { rc = make_map2(ctx, &mlk, (const __nv_bfloat16*)a.cache->lr_k + (size_t)a.agent * lr_rows * RK, lr_rows, RK, box_rows, C::RKP); if (rc) return rc; }
    if (RV) { rc = make_map2(ctx, &mlv, (const __nv_bfloat16*)a.cache->lr_v + (size_t)a.agent * lr_rows * RV, lr_rows, RV, box_rows, 64); if (rc) return rc; }
    PrefillTcParams p;
    p.q = (const __nv_bfloat16*)a.q; p.out = (__nv_bfloat16*)a.out; p.block_table = a.block_table;
    p.B_k = RK ? (const __nv_bfloat16*)a.B_k + (size_t)a.agent * RK * kvw : nullptr;
    p.B_v = RV ? (const __nv_bfloat16*)a.B_v + (size_t)a.agent * RV * kvw : nullptr;
    p.status = ctx->status; p.n_blocks = a.cache->n_blocks;
    p.S = a.S; p.T = a.T; p.first_block = a.first_block; p.contig = contig ? 1 : 0;
    p.longest_first = ctx->prefill_forward ? 0 : 1;
    p.n_q = d->n_q_heads; p.n_kv = d->n_kv_heads; p.group = G; p.tok_per_tile = PTC_TOK / G; p.k_stages = ks; p.v_stages = vs;
    p.scale_log2 = softmax_scale_log2(d); p.s_k = d->lora_scale_k; p.s_v = d->lora_scale_v;
    p.trace = (ctx->trace && ctx->trace_blocks >= 32) ? ctx->trace : nullptr;
    auto kern = lr_attend_prefill_tc_kernel<HD, RK, RV>;
    PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, smem));
    const int row_tiles = (a.S + p.tok_per_tile - 1) / p.tok_per_tile;
    // Short turn over a long context: too few (row tile, kv head) blocks to fill the machine, so the
    // context of each is split over a cluster of up to 8 blocks whose partial results merge over DSMEM.
    int ns = 1;
    const long long base_blocks = (long long)row_tiles * d->n_kv_heads;
    const int steps = (a.T + a.S + PTC_TOK - 1) / PTC_TOK;
    if (!ctx->no_prefill_split && C::SPLIT_BYTES <= C::Q_BYTES + C::QX_BYTES + ks * C::KSTAGE + vs * C::VSTAGE) {
      ns = (int)(ctx->sm_count / base_blocks);          // as many as keep the grid within one block per SM
      if (ns > 8) ns = 8;
      if (ns > steps / 8) ns = steps / 8;               // at least eight steps per block
      if (ns < 1) ns = 1;
      // every cluster must be resident at once (one block per SM, and a cluster lives inside one GPC): ask
      // the occupancy calculator once per cluster size, and shrink the clusters until the grid fits in one wave
      static int max_clusters_dev[kMaxDevices][9] = {{0}};   // 0 = unknown, else max active clusters + 1
      int* max_clusters = max_clusters_dev[ctx->device % kMaxDevices];
      while (ns > 1) {
        if (max_clusters[ns] == 0) {
          cudaLaunchConfig_t qc = {};
          qc.gridDim = dim3(1, 1, ns * (ctx->sm_count / ns)); qc.blockDim = dim3(PTC_THREADS); qc.dynamicSmemBytes = smem;
          cudaLaunchAttribute qa[1];
          qa[0].id = cudaLaunchAttributeClusterDimension;
          qa[0].val.clusterDim.x = 1; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = ns;
          qc.attrs = qa; qc.numAttrs = 1;
          int n = 0;
          if (cudaOccupancyMaxActiveClusters(&n, kern, &qc) != cudaSuccess) { cudaGetLastError(); n = 0; }
          max_clusters[ns] = n + 1;
        }
        if (max_clusters[ns] - 1 >= base_blocks) break;
        --ns;
      }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(row_tiles, d->n_kv_heads, ns);
    cfg.blockDim = dim3(PTC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = ns;
    cfg.attrs = attr; cfg.numAttrs = ns > 1 ? 1 : 0;
    PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, kern, mk, mv, mlk, mlv, p));
    return PRECC_OK;
  }
  static int32_t run(precc_ctx* ctx, const PrefillArgs& a) {
    if constexpr (PrefillTcCfg<HD, RK, RV>::supported) {
      const long long kv_rows = (long long)a.cache->n_blocks * a.d->n_kv_heads * PAGE;
      const bool aligned128 = ((reinterpret_cast<uintptr_t>(a.cache->k_base) | reinterpret_cast<uintptr_t>(a.cache->v_base) |
                                reinterpret_cast<uintptr_t>(a.cache->lr_k) | reinterpret_cast<uintptr_t>(a.cache->lr_v)) & 127u) == 0;
      if (kv_rows < (1ll << 31) && aligned128 && !ctx->force_simple_prefill) return run_tc(ctx, a);
    }
    return run_simple<false>(ctx, a);
  }
  // mma.sync kernel: oversized or unaligned caches, and the rotary variant
  template <bool ROPE = false>
  static int32_t run_simple(precc_ctx* ctx, const PrefillArgs& a) {
    using C = PrefillCfg<HD, RK, RV>;
    const precc_layer_desc* d = a.d;
    int stages = 3;
    while (stages > 2 && 2 * (C::smem_bytes(stages, ROPE) + 1024) > ctx->max_smem_optin) --stages;
    const int smem = C::smem_bytes(stages, ROPE);
    PrefillParams p;
    const size_t kvw = (size_t)d->n_kv_heads * HD;
    p.q = (const __nv_bfloat16*)a.q; p.out = (__nv_bfloat16*)a.out; p.block_table = a.block_table;
    p.k_base = (const __nv_bfloat16*)a.cache->k_base; p.v_base = (const __nv_bfloat16*)a.cache->v_base;
    p.lr_k = RK ? (const __nv_bfloat16*)a.cache->lr_k + (size_t)a.agent * a.cache->n_blocks * PAGE * RK : nullptr;
    p.lr_v = RV ? (const __nv_bfloat16*)a.cache->lr_v + (size_t)a.agent * a.cache->n_blocks * PAGE * RV : nullptr;
    p.B_k = RK ? (const __nv_bfloat16*)a.B_k + (size_t)a.agent * RK * kvw : nullptr;
    p.B_v = RV ? (const __nv_bfloat16*)a.B_v + (size_t)a.agent * RV * kvw : nullptr;
    p.status = ctx->status; p.n_blocks = a.cache->n_blocks;
    p.S = a.S; p.T = a.T; p.first_block = a.first_block;
    p.n_q = d->n_q_heads; p.n_kv = d->n_kv_heads; p.group = d->n_q_heads / d->n_kv_heads; p.stages = stages;
    p.scale_log2 = softmax_scale_log2(d); p.s_k = d->lora_scale_k; p.s_v = d->lora_scale_v;
    p.rope = reinterpret_cast<const float4*>(a.rope); p.max_pos = a.max_pos;
    auto kern = lr_attend_prefill_kernel<HD, RK, RV, ROPE>;
    PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, smem));
    const int row_tiles = (a.S * p.group + PF_ROWS - 1) / PF_ROWS;
    kern<<<dim3(row_tiles, d->n_kv_heads), PF_THREADS, smem, a.stream>>>(p);
    PRECC_CUDA(ctx, cudaGetLastError());
    return PRECC_OK;
  }
};

// Rotary keys: without a key-side adapter the rotated base cache is all there is (the position-free
// kernels are exact); with one, the mma.sync kernel expands and rotates the rank-r key term per tile.
template <int HD, int RK, int RV>
struct PrefillRunRope {
  static int32_t run(precc_ctx* ctx, const PrefillArgs& a) {
    if constexpr (RK > 0) return PrefillRun<HD, RK, RV>::template run_simple<true>(ctx, a);
    else return PrefillRun<HD, RK, RV>::run(ctx, a);
  }
};

struct CombineArgs {
  const precc_layer_desc* d; const float* recs; int n_shards; int B; const int32_t* agent_id; const void* B_v; void* out;
  cudaStream_t stream;
};
template <int HD, int RK, int RV>
struct CombineRun {
  static int32_t run(precc_ctx* ctx, const CombineArgs& a) {
    CombineParams p;
    p.recs = a.recs; p.agent_id = a.agent_id; p.B_v = (const __nv_bfloat16*)a.B_v; p.out = (__nv_bfloat16*)a.out;
    p.status = ctx->status; p.n_shards = a.n_shards; p.B = a.B;
    p.n_q = a.d->n_q_heads; p.n_kv = a.d->n_kv_heads; p.group = a.d->n_q_heads / a.d->n_kv_heads; p.n_agents = a.d->n_agents;
    p.s_v = a.d->lora_scale_v;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.d->n_kv_heads, a.B);
    cfg.blockDim = dim3(COMBINE_THREADS);
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, lr_combine_kernel<HD, RV>, p));
    return PRECC_OK;
  }
};

struct WsQuery { int sm_count, max_smem, B, n_kv, max_ctx; size_t* out; };
template <int HD, int RK, int RV>
struct DecodeWs {
  static int32_t run(precc_ctx*, const WsQuery& w) {
    *w.out = DecodeRun<HD, RK, RV>::ws_bytes(w.sm_count, w.max_smem, w.B, w.n_kv, w.max_ctx);
    return PRECC_OK;
  }
};

}  // namespace

// =========================================================================================== ABI
extern "C" {

int32_t precc_create(precc_ctx** out, int32_t device) {
  if (!out) return PRECC_ERR_INVALID_ARG;
  *out = nullptr;
  precc_ctx* ctx = new (std::nothrow) precc_ctx();
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  ctx->device = device;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->status, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMemset(ctx->status, 0, sizeof(uint32_t));
  if (e == cudaSuccess) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e == cudaSuccess && (qres != cudaDriverEntryPointSuccess || !fn)) e = cudaErrorUnknown;
    ctx->encode_tiled = reinterpret_cast<decltype(ctx->encode_tiled)>(fn);
  }
  if (const char* v = getenv("PRECC_PREFILL")) ctx->force_simple_prefill = (strcmp(v, "simple") == 0);
  if (const char* v = getenv("PRECC_GEMM")) ctx->force_tiled_gemm = (strcmp(v, "tiled") == 0);
  if (const char* v = getenv("PRECC_DEEP")) ctx->deep_clusters = (strcmp(v, "0") != 0);
  if (const char* v = getenv("PRECC_GEMM_SPLITK")) ctx->no_gemm_splitk = (strcmp(v, "0") == 0);
  if (const char* v = getenv("PRECC_DECODE")) ctx->force_ticket_decode = (strcmp(v, "ticket") == 0);
  if (const char* v = getenv("PRECC_PREFILL_ORDER")) ctx->prefill_forward = (strcmp(v, "forward") == 0);
  if (const char* v = getenv("PRECC_PREFILL_SPLIT")) ctx->no_prefill_split = (strcmp(v, "0") == 0);
  if (e != cudaSuccess) {
    fprintf(stderr, "precc_create: %s\n", cudaGetErrorString(e));
    if (ctx->status) cudaFree(ctx->status);
    delete ctx;
    return PRECC_ERR_CUDA;
  }
  *out = ctx;
  return PRECC_OK;
}

int32_t precc_destroy(precc_ctx* ctx) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (ctx->status) cudaFree(ctx->status);
  delete ctx;
  return PRECC_OK;
}

const char* precc_last_error(const precc_ctx* ctx) { return ctx ? ctx->err : "null context"; }

const char* precc_error_name(int32_t code) {
  switch (code) {
    case PRECC_OK: return "PRECC_OK";
    case PRECC_ERR_INVALID_ARG: return "PRECC_ERR_INVALID_ARG";
    case PRECC_ERR_UNSUPPORTED: return "PRECC_ERR_UNSUPPORTED";
    case PRECC_ERR_MISALIGNED: return "PRECC_ERR_MISALIGNED";
    case PRECC_ERR_WORKSPACE: return "PRECC_ERR_WORKSPACE";
    case PRECC_ERR_CUDA: return "PRECC_ERR_CUDA";
    case PRECC_ERR_DEVICE_STATUS: return "PRECC_ERR_DEVICE_STATUS";
    default: return "PRECC_ERR_?";
  }
}

int32_t precc_sm_count(const precc_ctx* ctx) { return ctx ? ctx->sm_count : 0; }

int32_t precc_set_trace_buffer(precc_ctx* ctx, void* buffer, size_t n_blocks) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (buffer && (reinterpret_cast<uintptr_t>(buffer) & 7u)) return fail(ctx, PRECC_ERR_MISALIGNED, "trace buffer not 8-byte aligned");
  ctx->trace = static_cast<unsigned long long*>(buffer);
  ctx->trace_blocks = buffer ? n_blocks : 0;
  return PRECC_OK;
}

int32_t precc_poll_status(precc_ctx* ctx, void* stream, uint32_t* status_out) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t h = 0;
  PRECC_CUDA(ctx, cudaMemcpyAsync(&h, ctx->status, sizeof(h), cudaMemcpyDeviceToHost, st));
  PRECC_CUDA(ctx, cudaMemsetAsync(ctx->status, 0, sizeof(h), st));
  PRECC_CUDA(ctx, cudaStreamSynchronize(st));
  if (status_out) *status_out = h;
  if (h) return fail(ctx, PRECC_ERR_DEVICE_STATUS, "device status 0x%x%s%s", h, (h & PRECC_STATUS_BAD_INDEX) ? " bad-index" : "",
                     (h & PRECC_STATUS_TIMEOUT) ? " timeout" : "");
  return PRECC_OK;
}

int32_t precc_pack_kmajor(precc_ctx* ctx, const void* src, int32_t d_model, int32_t n_cols, void* dst, int32_t dst_rows,
                          int32_t dst_row0, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (n_cols == 0) return PRECC_OK;
  if (!src || !dst || d_model <= 0 || n_cols < 0 || dst_row0 < 0 || dst_row0 + n_cols > dst_rows)
    return fail(ctx, PRECC_ERR_INVALID_ARG, "pack_kmajor: bad arguments");
  if (d_model % GEMM_BK) return fail(ctx, PRECC_ERR_UNSUPPORTED, "pack_kmajor: d_model %% 64 != 0");
  dim3 grid((n_cols + 31) / 32, (d_model + 31) / 32), block(32, 8);
  pack_kmajor_kernel<<<grid, block, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)src, d_model, n_cols, (__nv_bfloat16*)dst, dst_rows, dst_row0);
  PRECC_CUDA(ctx, cudaGetLastError());
  return PRECC_OK;
}

int32_t precc_lr_precompute(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* A_packed,
                            const int32_t* slot_mapping, int64_t start_slot, uint64_t agent_mask, const precc_cache* cache,
                            void* stream) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (M < 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "M < 0");
  const int n_out = desc->n_agents * (desc->rank_k + desc->rank_v);
  if (M == 0 || n_out == 0) return PRECC_OK;
  rc = check_cache(ctx, desc, cache, false, true);
  if (rc) return rc;
  if (!H || !A_packed) return fail(ctx, PRECC_ERR_INVALID_ARG, "H or A_packed is null");
  if (!aligned16(H) || !aligned16(A_packed)) return fail(ctx, PRECC_ERR_MISALIGNED, "H / A_packed not 16-byte aligned");
  if (!slot_mapping && (start_slot < 0 || start_slot + M > cache->n_blocks * PRECC_PAGE))
    return fail(ctx, PRECC_ERR_INVALID_ARG, "slots [%lld, %lld) outside the cache", (long long)start_slot, (long long)start_slot + M);
  GemmParams gp{};
  gp.mode = 0; gp.slot_mapping = slot_mapping; gp.start_slot = start_slot; gp.n_blocks = cache->n_blocks;
  gp.lr_k = (__nv_bfloat16*)cache->lr_k; gp.lr_v = (__nv_bfloat16*)cache->lr_v;
  gp.n_agents = desc->n_agents; gp.rank_k = desc->rank_k; gp.rank_v = desc->rank_v; gp.agent_mask = agent_mask;
  gp.n_kv = desc->n_kv_heads; gp.hd = desc->head_dim;
  return launch_gemm(ctx, H, M, desc->d_model, A_packed, n_out, gp, (cudaStream_t)stream);
}

static int32_t set_rope(precc_ctx* ctx, const precc_layer_desc* desc, const precc_rope* rope, GemmParams* gp) {
  if (!rope) return PRECC_OK;
  if (!rope->table || rope->max_pos < 1) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table is null or empty");
  if (!aligned16(rope->table)) return fail(ctx, PRECC_ERR_MISALIGNED, "rope table not 16-byte aligned");
  if (!rope->positions && (rope->start_pos < 0 || rope->start_pos + gp->M > rope->max_pos))
    return fail(ctx, PRECC_ERR_INVALID_ARG, "positions [%lld, %lld) outside the rope table", (long long)rope->start_pos,
                (long long)rope->start_pos + gp->M);
  (void)desc;
  gp->rope = reinterpret_cast<const float4*>(rope->table); gp->positions = rope->positions;
  gp->start_pos = rope->start_pos; gp->max_pos = rope->max_pos;
  return PRECC_OK;
}

static int32_t rebase_entry(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* W_packed,
                            const int32_t* slot_mapping, int64_t start_slot, const precc_rope* rope, const precc_cache* cache,
                            void* stream) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (M < 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "M < 0");
  if (M == 0) return PRECC_OK;
  rc = check_cache(ctx, desc, cache, true, false);
  if (rc) return rc;
  if (!H || !W_packed) return fail(ctx, PRECC_ERR_INVALID_ARG, "H or W_packed is null");
  if (!aligned16(H) || !aligned16(W_packed)) return fail(ctx, PRECC_ERR_MISALIGNED, "H / W_packed not 16-byte aligned");
  if (!slot_mapping && (start_slot < 0 || start_slot + M > cache->n_blocks * PRECC_PAGE))
    return fail(ctx, PRECC_ERR_INVALID_ARG, "slots [%lld, %lld) outside the cache", (long long)start_slot, (long long)start_slot + M);
  GemmParams gp{};
  gp.mode = 1; gp.slot_mapping = slot_mapping; gp.start_slot = start_slot; gp.n_blocks = cache->n_blocks;
  gp.base_k = (__nv_bfloat16*)cache->k_base; gp.base_v = (__nv_bfloat16*)cache->v_base;
  gp.n_agents = desc->n_agents; gp.rank_k = desc->rank_k; gp.rank_v = desc->rank_v; gp.agent_mask = ~0ull;
  gp.n_kv = desc->n_kv_heads; gp.hd = desc->head_dim;
  gp.M = M;
  rc = set_rope(ctx, desc, rope, &gp);
  if (rc) return rc;
  return launch_gemm(ctx, H, M, desc->d_model, W_packed, 2 * desc->n_kv_heads * desc->head_dim, gp, (cudaStream_t)stream);
}

int32_t precc_rebase_project(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* W_packed,
                             const int32_t* slot_mapping, int64_t start_slot, const precc_cache* cache, void* stream) {
  return rebase_entry(ctx, desc, H, M, W_packed, slot_mapping, start_slot, nullptr, cache, stream);
}

int32_t precc_rebase_project_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* W_packed,
                                  const int32_t* slot_mapping, int64_t start_slot, const precc_rope* rope,
                                  const precc_cache* cache, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!rope) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope is null");
  return rebase_entry(ctx, desc, H, M, W_packed, slot_mapping, start_slot, rope, cache, stream);
}

static int32_t turn_entry(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* WA_packed,
                          const int32_t* slot_mapping, int64_t start_slot, uint64_t agent_mask, const precc_rope* rope,
                          const precc_cache* cache, void* stream, const uint64_t* row_masks = nullptr) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (M < 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "M < 0");
  if (M == 0) return PRECC_OK;
  const int n_lr = desc->n_agents * (desc->rank_k + desc->rank_v);
  rc = check_cache(ctx, desc, cache, true, n_lr > 0);
  if (rc) return rc;
  if (!H || !WA_packed) return fail(ctx, PRECC_ERR_INVALID_ARG, "H or WA_packed is null");
  if (!aligned16(H) || !aligned16(WA_packed)) return fail(ctx, PRECC_ERR_MISALIGNED, "H / WA_packed not 16-byte aligned");
  if (!slot_mapping && (start_slot < 0 || start_slot + M > cache->n_blocks * PRECC_PAGE))
    return fail(ctx, PRECC_ERR_INVALID_ARG, "slots [%lld, %lld) outside the cache", (long long)start_slot, (long long)start_slot + M);
  GemmParams gp{};
  gp.mode = 2; gp.slot_mapping = slot_mapping; gp.start_slot = start_slot; gp.n_blocks = cache->n_blocks;
  gp.base_k = (__nv_bfloat16*)cache->k_base; gp.base_v = (__nv_bfloat16*)cache->v_base;
  gp.lr_k = (__nv_bfloat16*)cache->lr_k; gp.lr_v = (__nv_bfloat16*)cache->lr_v;
  gp.n_agents = desc->n_agents; gp.rank_k = desc->rank_k; gp.rank_v = desc->rank_v; gp.agent_mask = agent_mask;
  gp.row_masks = reinterpret_cast<const unsigned long long*>(row_masks);
  gp.n_kv = desc->n_kv_heads; gp.hd = desc->head_dim;
  gp.M = M;
  rc = set_rope(ctx, desc, rope, &gp);
  if (rc) return rc;
  return launch_gemm(ctx, H, M, desc->d_model, WA_packed, 2 * desc->n_kv_heads * desc->head_dim + n_lr, gp, (cudaStream_t)stream);
}

int32_t precc_turn_project(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* WA_packed,
                           const int32_t* slot_mapping, int64_t start_slot, uint64_t agent_mask, const precc_cache* cache,
                           void* stream) {
  return turn_entry(ctx, desc, H, M, WA_packed, slot_mapping, start_slot, agent_mask, nullptr, cache, stream);
}

int32_t precc_turn_project_rows(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* WA_packed,
                                const int32_t* slot_mapping, const uint64_t* row_agent_masks, const precc_cache* cache,
                                void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!slot_mapping || !row_agent_masks) return fail(ctx, PRECC_ERR_INVALID_ARG, "slot_mapping / row_agent_masks is null");
  if (reinterpret_cast<uintptr_t>(row_agent_masks) & 7u) return fail(ctx, PRECC_ERR_MISALIGNED, "row_agent_masks not 8-byte aligned");
  return turn_entry(ctx, desc, H, M, WA_packed, slot_mapping, 0, 0, nullptr, cache, stream, row_agent_masks);
}

int32_t precc_turn_project_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* WA_packed,
                                const int32_t* slot_mapping, int64_t start_slot, uint64_t agent_mask, const precc_rope* rope,
                                const precc_cache* cache, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!rope) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope is null");
  return turn_entry(ctx, desc, H, M, WA_packed, slot_mapping, start_slot, agent_mask, rope, cache, stream);
}

size_t precc_decode_workspace_bytes(const precc_layer_desc* desc, int32_t max_batch, int32_t max_ctx, int32_t sm_count) {
  if (!desc || max_batch <= 0 || max_ctx <= 0 || sm_count <= 0) return 0;
  size_t out = 0;
  // the ring depth depends on the opt-in shared memory of the device; sm_100 offers 227 KB
  WsQuery w{sm_count, 232448, max_batch, desc->n_kv_heads, max_ctx, &out};
  precc_ctx tmp;
  if (dispatch_shape<DecodeWs>(&tmp, desc->head_dim, desc->rank_k, desc->rank_v, w) != PRECC_OK) return 0;
  return out;
}

int32_t precc_workspace_init(precc_ctx* ctx, void* workspace, size_t workspace_bytes, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes == 0) return fail(ctx, PRECC_ERR_WORKSPACE, "workspace is null or empty");
  PRECC_CUDA(ctx, cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream));
  return PRECC_OK;
}

static int32_t decode_entry(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B, const int32_t* agent_id,
                            const int32_t* ctx_len, const int32_t* block_table, int32_t table_stride,
                            const int32_t* first_block, int32_t max_ctx, const void* B_k, const void* B_v,
                            const precc_cache* cache, void* out, void* workspace, size_t workspace_bytes, void* stream,
                            const float* rope, int32_t max_pos, float* raw = nullptr) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (B < 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "B < 0");
  if (B == 0) return PRECC_OK;
  rc = check_cache(ctx, desc, cache, true, true);
  if (rc) return rc;
  if (!q || !out || !agent_id || !ctx_len) return fail(ctx, PRECC_ERR_INVALID_ARG, "q / out / agent_id / ctx_len is null");
  if ((desc->rank_k > 0 && !B_k) || (desc->rank_v > 0 && !B_v && !raw)) return fail(ctx, PRECC_ERR_INVALID_ARG, "B_k / B_v is null");
  if (!aligned16(q) || !aligned16(out) || !aligned16(B_k) || !aligned16(B_v) || !aligned16(workspace))
    return fail(ctx, PRECC_ERR_MISALIGNED, "q / out / B_k / B_v / workspace not 16-byte aligned");
  if (max_ctx < 1) return fail(ctx, PRECC_ERR_INVALID_ARG, "max_ctx < 1");
  if (block_table && (long long)table_stride * PRECC_PAGE < max_ctx)
    return fail(ctx, PRECC_ERR_INVALID_ARG, "block table stride %d too short for max_ctx %d", table_stride, max_ctx);
  if (B > 65535) return fail(ctx, PRECC_ERR_UNSUPPORTED, "B > 65535");
  if (ctx->max_smem_optin != 232448) {
    // the workspace query assumes the sm_100 shared-memory size
    return fail(ctx, PRECC_ERR_UNSUPPORTED, "device opt-in shared memory %d != 232448 (not an sm_100 part?)", ctx->max_smem_optin);
  }
  DecodeArgs a{desc, q, B, agent_id, ctx_len, block_table, table_stride, first_block, max_ctx, B_k, B_v, cache, out,
               workspace, workspace_bytes, (cudaStream_t)stream};
  a.raw = raw;
  if (!rope) return dispatch_shape<DecodeRun>(ctx, desc->head_dim, desc->rank_k, desc->rank_v, a);
  if (raw) return fail(ctx, PRECC_ERR_UNSUPPORTED, "partial records with rotary keys");   // compiled out of the rotary kernels
  if (!aligned16(rope)) return fail(ctx, PRECC_ERR_MISALIGNED, "rope table not 16-byte aligned");
  if (max_pos < max_ctx) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table covers %d positions, max_ctx is %d", max_pos, max_ctx);
  a.rope = rope; a.max_pos = max_pos;
  return dispatch_shape<DecodeRunRope>(ctx, desc->head_dim, desc->rank_k, desc->rank_v, a);
}

int32_t precc_lr_attend_decode(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B, const int32_t* agent_id,
                               const int32_t* ctx_len, const int32_t* block_table, int32_t table_stride,
                               const int32_t* first_block, int32_t max_ctx, const void* B_k, const void* B_v,
                               const precc_cache* cache, void* out, void* workspace, size_t workspace_bytes, void* stream) {
  return decode_entry(ctx, desc, q, B, agent_id, ctx_len, block_table, table_stride, first_block, max_ctx, B_k, B_v, cache, out,
                      workspace, workspace_bytes, stream, nullptr, 0);
}

int32_t precc_lr_attend_decode_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                                    const int32_t* agent_id, const int32_t* ctx_len, const int32_t* block_table,
                                    int32_t table_stride, const int32_t* first_block, int32_t max_ctx, const void* B_k,
                                    const void* B_v, const precc_rope* rope, const precc_cache* cache, void* out,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!rope || !rope->table) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table is null");
  return decode_entry(ctx, desc, q, B, agent_id, ctx_len, block_table, table_stride, first_block, max_ctx, B_k, B_v, cache, out,
                      workspace, workspace_bytes, stream, rope->table, rope->max_pos);
}

size_t precc_partial_record_floats(const precc_layer_desc* desc) {
  if (!desc) return 0;
  return (size_t)16 + 8 * (size_t)(desc->head_dim + desc->rank_v);
}

int32_t precc_lr_attend_decode_partial(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                                       const int32_t* agent_id, const int32_t* ctx_len, const int32_t* block_table,
                                       int32_t table_stride, const int32_t* first_block, int32_t max_ctx, const void* B_k,
                                       const precc_cache* cache, float* records, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!records || !aligned16(records)) return fail(ctx, PRECC_ERR_INVALID_ARG, "records is null or not 16-byte aligned");
  // `out` is not written in this mode (the records pointer stands in for it); B_v is not needed: the
  // value-side epilogue belongs to the combine step
  return decode_entry(ctx, desc, q, B, agent_id, ctx_len, block_table, table_stride, first_block, max_ctx, B_k, nullptr, cache,
                      records, workspace, workspace_bytes, stream, nullptr, 0, records);
}

int32_t precc_combine_partials(precc_ctx* ctx, const precc_layer_desc* desc, const float* records, int32_t n_shards, int32_t B,
                               const int32_t* agent_id, const void* B_v, void* out, void* stream) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (B < 0 || n_shards < 1 || n_shards > 64) return fail(ctx, PRECC_ERR_INVALID_ARG, "B < 0 or n_shards outside [1, 64]");
  if (B == 0) return PRECC_OK;
  if (!records || !agent_id || !out) return fail(ctx, PRECC_ERR_INVALID_ARG, "records / agent_id / out is null");
  if (desc->rank_v > 0 && !B_v) return fail(ctx, PRECC_ERR_INVALID_ARG, "B_v is null");
  if (!aligned16(records) || !aligned16(out) || !aligned16(B_v)) return fail(ctx, PRECC_ERR_MISALIGNED, "records / out / B_v not 16-byte aligned");
  if (B > 65535) return fail(ctx, PRECC_ERR_UNSUPPORTED, "B > 65535");
  CombineArgs a{desc, records, n_shards, B, agent_id, B_v, out, (cudaStream_t)stream};
  return dispatch_shape<CombineRun>(ctx, desc->head_dim, desc->rank_k, desc->rank_v, a);
}

int32_t precc_lr_attend_decode_static(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                                      const int32_t* agent_id, const int32_t* ctx_len, const int32_t* block_table,
                                      int32_t table_stride, const int32_t* first_block, int32_t max_ctx, const void* B_k,
                                      const void* B_v, const precc_cache* cache, void* out, void* stream) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (B < 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "B < 0");
  if (B == 0) return PRECC_OK;
  if (max_ctx < 1) return fail(ctx, PRECC_ERR_INVALID_ARG, "max_ctx < 1");
  const size_t need = precc_decode_workspace_bytes(desc, B, max_ctx, ctx->sm_count);
  if (need == 0) return fail(ctx, PRECC_ERR_UNSUPPORTED, "no decode kernel for this shape");
  if (need > PRECC_STATIC_SCRATCH_BYTES)
    return fail(ctx, PRECC_ERR_WORKSPACE, "this call needs %zu bytes of scratch but the built-in array holds %u; "
                "use precc_lr_attend_decode with a caller workspace", need, (unsigned)PRECC_STATIC_SCRATCH_BYTES);
  if (ctx->device < 0 || ctx->device >= kMaxDevices) return fail(ctx, PRECC_ERR_UNSUPPORTED, "device index %d >= %d", ctx->device, kMaxDevices);
  void* scratch = g_static_scratch_addr[ctx->device];
  if (!scratch) {
    // once per device, with that device current: the symbol's address differs from GPU to GPU
    int cur = -1;
    PRECC_CUDA(ctx, cudaGetDevice(&cur));
    if (cur != ctx->device) return fail(ctx, PRECC_ERR_INVALID_ARG, "current device %d is not the context's device %d", cur, ctx->device);
    PRECC_CUDA(ctx, cudaGetSymbolAddress(&scratch, g_static_scratch));
    g_static_scratch_addr[ctx->device] = scratch;
  }
  // the arrival counters at the head of the scratch must be zero when the kernel starts
  const size_t counters = ((size_t)B * desc->n_kv_heads * 4 + 255) / 256 * 256;
  PRECC_CUDA(ctx, cudaMemsetAsync(scratch, 0, counters, (cudaStream_t)stream));
  return precc_lr_attend_decode(ctx, desc, q, B, agent_id, ctx_len, block_table, table_stride, first_block, max_ctx, B_k, B_v,
                                cache, out, scratch, PRECC_STATIC_SCRATCH_BYTES, stream);
}

static int32_t prefill_entry(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S, int32_t agent,
                             int32_t ctx_len, const int32_t* block_table, int32_t table_stride, int32_t first_block,
                             const void* B_k, const void* B_v, const precc_rope* rope, const precc_cache* cache, void* out,
                             void* stream) {
  int32_t rc = check_desc(ctx, desc);
  if (rc) return rc;
  if (S < 0 || ctx_len < 0) return fail(ctx, PRECC_ERR_INVALID_ARG, "S < 0 or ctx_len < 0");
  if (S == 0) return PRECC_OK;
  rc = check_cache(ctx, desc, cache, true, true);
  if (rc) return rc;
  if (!q || !out) return fail(ctx, PRECC_ERR_INVALID_ARG, "q / out is null");
  if (agent < -1 || agent >= desc->n_agents) return fail(ctx, PRECC_ERR_INVALID_ARG, "agent %d outside [-1,%d)", agent, desc->n_agents);
  const bool neutral = agent < 0;       // adapter-free view: base cache only
  if (!neutral && ((desc->rank_k > 0 && !B_k) || (desc->rank_v > 0 && !B_v))) return fail(ctx, PRECC_ERR_INVALID_ARG, "B_k / B_v is null");
  if (!aligned16(q) || !aligned16(out) || !aligned16(B_k) || !aligned16(B_v)) return fail(ctx, PRECC_ERR_MISALIGNED, "q / out / B_k / B_v not 16-byte aligned");
  const long long need_blocks = ((long long)ctx_len + S + PRECC_PAGE - 1) / PRECC_PAGE;
  if (block_table && table_stride < need_blocks) return fail(ctx, PRECC_ERR_INVALID_ARG, "block table has %d entries, need %lld", table_stride, need_blocks);
  if (!block_table && (first_block < 0 || first_block + need_blocks > cache->n_blocks))
    return fail(ctx, PRECC_ERR_INVALID_ARG, "blocks [%d, %lld) outside the cache", first_block, first_block + need_blocks);
  if ((long long)S * (desc->n_q_heads / desc->n_kv_heads) > (long long)PF_ROWS * 65535) return fail(ctx, PRECC_ERR_UNSUPPORTED, "S too large");
  PrefillArgs a{desc, q, S, neutral ? 0 : agent, ctx_len, block_table, first_block, B_k, B_v, cache, out, (cudaStream_t)stream};
  if (!rope) return dispatch_shape<PrefillRun>(ctx, desc->head_dim, neutral ? 0 : desc->rank_k, neutral ? 0 : desc->rank_v, a);
  if (!rope->table || !aligned16(rope->table)) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table is null or not 16-byte aligned");
  if ((long long)rope->max_pos < (long long)ctx_len + S)
    return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table covers %d positions, the turn ends at %lld", rope->max_pos, (long long)ctx_len + S);
  a.rope = rope->table; a.max_pos = rope->max_pos;
  return dispatch_shape<PrefillRunRope>(ctx, desc->head_dim, neutral ? 0 : desc->rank_k, neutral ? 0 : desc->rank_v, a);
}

int32_t precc_lr_attend_prefill(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S, int32_t agent,
                                int32_t ctx_len, const int32_t* block_table, int32_t table_stride, int32_t first_block,
                                const void* B_k, const void* B_v, const precc_cache* cache, void* out, void* stream) {
  return prefill_entry(ctx, desc, q, S, agent, ctx_len, block_table, table_stride, first_block, B_k, B_v, nullptr, cache, out, stream);
}

int32_t precc_lr_attend_prefill_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S, int32_t agent,
                                     int32_t ctx_len, const int32_t* block_table, int32_t table_stride, int32_t first_block,
                                     const void* B_k, const void* B_v, const precc_rope* rope, const precc_cache* cache,
                                     void* out, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!rope) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope is null");
  return prefill_entry(ctx, desc, q, S, agent, ctx_len, block_table, table_stride, first_block, B_k, B_v, rope, cache, out, stream);
}

}  // extern "C"
