// libprecc: context life cycle, error plumbing, argument checks, tensor-map helpers, weight packing.
#include "api_internal.h"
#include "tc_common.cuh"

namespace precc {

int32_t fail(precc_ctx* ctx, int32_t code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

namespace {
struct SmemLimit { const void* fn; int dev; int bytes; };
std::mutex g_limits_mu;
SmemLimit g_limits[1024];
int g_n_limits = 0;
}  // namespace

cudaError_t raise_smem_limit_raw(precc_ctx* ctx, const void* fn, int bytes) {
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

std::recursive_mutex& lazy_mu() {
  static std::recursive_mutex mu;
  return mu;
}

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

// ------------------------------------------------------------------------------------ tensor maps
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


namespace {
// A barrier that nothing ever arrives on: the waiting lane must give up after the context's wait limit, record
// PRECC_STATUS_TIMEOUT and let the kernel end normally (the self-test of the bounded waits every tcgen05 / TMA
// kernel of the library uses).
__global__ void wait_timeout_selftest_kernel(uint32_t* status, uint32_t* done_flag) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&bar), 0, status);
  __syncwarp();
  if (threadIdx.x == 0) *done_flag = ok ? 1u : 2u;      // 2: the wait expired and the kernel carried on to its end
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

}  // namespace

}  // namespace precc

using namespace precc;

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
  if (e == cudaSuccess) e = cudaMalloc(&ctx->status, 2 * sizeof(uint32_t));
  if (e == cudaSuccess) {
    const uint32_t init[2] = {0u, kDefaultWaitLimit};
    e = cudaMemcpy(ctx->status, init, sizeof(init), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e == cudaSuccess && (qres != cudaDriverEntryPointSuccess || !fn)) e = cudaErrorUnknown;
    ctx->encode_tiled = reinterpret_cast<decltype(ctx->encode_tiled)>(fn);
  }
  if (const char* v = getenv("PRECC_PREFILL")) ctx->force_simple_prefill = (strcmp(v, "simple") == 0);
  if (const char* v = getenv("PRECC_GEMM")) { ctx->force_tiled_gemm = (strcmp(v, "tiled") == 0); ctx->gemm_pair = (strcmp(v, "pair") == 0); }
  if (const char* v = getenv("PRECC_DEEP")) { ctx->deep_clusters = (strcmp(v, "0") != 0); ctx->deep_always = (strcmp(v, "2") == 0); }
  if (const char* v = getenv("PRECC_DECODE_CLUSTER")) ctx->decode_cluster_cap = atoi(v);
  if (const char* v = getenv("PRECC_DECODE_POLICY")) ctx->decode_cluster_policy = atoi(v);
  if (const char* v = getenv("PRECC_DECODE_STAGES")) ctx->decode_stage_cap = atoi(v);
  if (const char* v = getenv("PRECC_DECODE_PRE")) ctx->decode_pre_stages = atoi(v);
  if (const char* v = getenv("PRECC_GEMM_STAGES")) ctx->gemm_stage_cap = atoi(v);
  if (const char* v = getenv("PRECC_GEMM_KS_MAX")) ctx->gemm_ks_max = atoi(v);
  if (const char* v = getenv("PRECC_GEMM_DIRECT")) ctx->gemm_direct = atoi(v);
  if (const char* v = getenv("PRECC_GEMM_PUSH_MAX")) ctx->gemm_push_max = atoi(v);
  if (const char* v = getenv("PRECC_GEMM_KS_MIN")) { ctx->gemm_ks_min = atoi(v); if (ctx->gemm_ks_min < 2) ctx->gemm_ks_min = 2; }
  if (const char* v = getenv("PRECC_GEMM_SPLITK")) ctx->no_gemm_splitk = (strcmp(v, "0") == 0);
  if (const char* v = getenv("PRECC_DECODE")) ctx->force_ticket_decode = (strcmp(v, "ticket") == 0);
  if (const char* v = getenv("PRECC_PREFILL_ORDER")) ctx->prefill_forward = (strcmp(v, "forward") == 0);
  if (const char* v = getenv("PRECC_PREFILL_SPLIT")) ctx->no_prefill_split = (strcmp(v, "0") == 0);
  if (const char* v = getenv("PRECC_PREFILL_VHALF")) ctx->no_prefill_vhalf = (strcmp(v, "0") == 0);
  if (const char* v = getenv("PRECC_PREFILL_HELPERS")) ctx->no_prefill_helpers = (strcmp(v, "0") == 0);
  if (const char* v = getenv("PRECC_PREFILL_HELPER_P")) ctx->prefill_helper_p = atoi(v);
  if (const char* v = getenv("PRECC_PREFILL_HELPER_MIN")) { const int n = atoi(v); if (n >= 8) ctx->prefill_helper_min_steps = n; }
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

int32_t precc_set_wait_limit(precc_ctx* ctx, uint64_t sm_cycles) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  uint64_t units = sm_cycles == 0 ? kDefaultWaitLimit : (sm_cycles + 1023) >> 10;
  if (units > 0xffffffffull) units = 0xffffffffull;
  const uint32_t v = static_cast<uint32_t>(units < 1 ? 1 : units);
  PRECC_CUDA(ctx, cudaMemcpy(ctx->status + 1, &v, sizeof(v), cudaMemcpyHostToDevice));
  return PRECC_OK;
}

int32_t precc_selftest_wait_timeout(precc_ctx* ctx, uint32_t* done_flag, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!done_flag) return fail(ctx, PRECC_ERR_INVALID_ARG, "done_flag is null");
  wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->status, done_flag);
  PRECC_CUDA(ctx, cudaGetLastError());
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

}  // extern "C"
