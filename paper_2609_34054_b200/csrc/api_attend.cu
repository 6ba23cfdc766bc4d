// libprecc: the attention entry points (decode, its rotary, partial-record and allocation-free forms, the
// combine step of context-sharded decode, new-turn prefill).  The kernels themselves are compiled in the
// per-head-dimension units; this file validates arguments and forwards.
#include "api_internal.h"
#include "combine.cuh"
#include "prefill.cuh"   // PF_ROWS (the size check of the prefill entry)
#include "rope_expand.cuh"

using namespace precc;

// Scratch for precc_lr_attend_decode_static: lives in the library image, one copy per GPU that loads it.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[PRECC_STATIC_SCRATCH_BYTES];

namespace {

// Device address of g_static_scratch on each device, looked up on the first static call there.
void* g_static_scratch_addr[kMaxDevices] = {nullptr};

int32_t decode_run(precc_ctx* ctx, const DecodeArgs& a) {
  return a.d->head_dim == 64 ? decode_run_hd64(ctx, a) : decode_run_hd128(ctx, a);
}

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

}  // namespace

extern "C" {

size_t precc_decode_workspace_bytes(const precc_layer_desc* desc, int32_t max_batch, int32_t max_ctx, int32_t sm_count) {
  if (!desc || max_batch <= 0 || max_ctx <= 0 || sm_count <= 0) return 0;
  size_t out = 0;
  // the ring depth depends on the opt-in shared memory of the device; sm_100 offers 227 KB
  WsQuery w{sm_count, 232448, max_batch, desc->n_kv_heads, max_ctx, &out};
  precc_ctx tmp;
  if (desc->head_dim != 64 && desc->head_dim != 128) return 0;
  const int32_t rc = desc->head_dim == 64 ? decode_ws_hd64(&tmp, desc->rank_k, desc->rank_v, w)
                                          : decode_ws_hd128(&tmp, desc->rank_k, desc->rank_v, w);
  return rc == PRECC_OK ? out : 0;
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
                            const float* rope, int32_t max_pos, float* raw = nullptr, bool clear_counters = false) {
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
  a.clear_counters = clear_counters;
  if (!rope) return decode_run(ctx, a);
  if (raw) return fail(ctx, PRECC_ERR_UNSUPPORTED, "partial records with rotary keys");   // compiled out of the rotary kernels
  if (!aligned16(rope)) return fail(ctx, PRECC_ERR_MISALIGNED, "rope table not 16-byte aligned");
  if (max_pos < max_ctx) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table covers %d positions, max_ctx is %d", max_pos, max_ctx);
  a.rope = rope; a.max_pos = max_pos;
  return decode_run(ctx, a);
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
  return desc->head_dim == 64 ? dispatch_ranks<CombineRun, 64>(ctx, desc->rank_k, desc->rank_v, a)
                              : dispatch_ranks<CombineRun, 128>(ctx, desc->rank_k, desc->rank_v, a);
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
  void* scratch = nullptr;
  {
    std::lock_guard<std::recursive_mutex> lk(lazy_mu());
    scratch = g_static_scratch_addr[ctx->device];
    if (!scratch) {
      // once per device, with that device current: the symbol's address differs from GPU to GPU
      int cur = -1;
      PRECC_CUDA(ctx, cudaGetDevice(&cur));
      if (cur != ctx->device) return fail(ctx, PRECC_ERR_INVALID_ARG, "current device %d is not the context's device %d", cur, ctx->device);
      PRECC_CUDA(ctx, cudaGetSymbolAddress(&scratch, g_static_scratch));
      g_static_scratch_addr[ctx->device] = scratch;
    }
  }
  // The arrival counters at the head of the scratch must be zero when the kernel that uses them starts: they are
  // cleared on the stream right before that launch, i.e. only after every argument check has passed and only when
  // the split schedule really takes the kernel that merges through the scratch.
  return decode_entry(ctx, desc, q, B, agent_id, ctx_len, block_table, table_stride, first_block, max_ctx, B_k, B_v, cache, out,
                      scratch, PRECC_STATIC_SCRATCH_BYTES, stream, nullptr, 0, nullptr, /*clear_counters=*/true);
}

static int32_t prefill_entry(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S, int32_t agent,
                             int32_t ctx_len, const int32_t* block_table, int32_t table_stride, int32_t first_block,
                             const void* B_k, const void* B_v, const precc_rope* rope, const precc_cache* cache, void* out,
                             void* stream, void* k_scratch = nullptr, size_t k_scratch_bytes = 0, void* ws = nullptr,
                             size_t ws_bytes = 0) {
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
  if (ws) {
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return fail(ctx, PRECC_ERR_MISALIGNED, "prefill workspace not 256-byte aligned");
    a.ws = ws; a.ws_bytes = ws_bytes;
  }
  const int rk = neutral ? 0 : desc->rank_k, rv = neutral ? 0 : desc->rank_v;
  auto run = [&]() { return desc->head_dim == 64 ? prefill_run_hd64(ctx, a, rk, rv) : prefill_run_hd128(ctx, a, rk, rv); };
  if (!rope) return run();
  if (!rope->table || !aligned16(rope->table)) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table is null or not 16-byte aligned");
  if ((long long)rope->max_pos < (long long)ctx_len + S)
    return fail(ctx, PRECC_ERR_INVALID_ARG, "rope table covers %d positions, the turn ends at %lld", rope->max_pos, (long long)ctx_len + S);
  a.rope = rope->table; a.max_pos = rope->max_pos;
  if (!k_scratch || rk == 0) return run();     // no key-side adapter in play: the rotated base cache is all there is
  // Rotary prefill with scratch: write the adapted rotary keys of the sequence out once (logical block order), then run
  // the tensor-memory kernel on them without a key-side adapter.  Falls back to the per-tile expansion of the
  // mma.sync kernel where the tensor-memory kernel does not take the call.
  const long long stage_blocks = 128 / PRECC_PAGE;            // whole 128-token stages of the tensor-memory kernel
  const long long out_blocks = (need_blocks + stage_blocks - 1) / stage_blocks * stage_blocks;
  const size_t need_bytes = (size_t)out_blocks * desc->n_kv_heads * PRECC_PAGE * desc->head_dim * 2;
  if (k_scratch_bytes < need_bytes) return fail(ctx, PRECC_ERR_WORKSPACE, "key scratch: need %zu bytes, got %zu", need_bytes, k_scratch_bytes);
  if ((reinterpret_cast<uintptr_t>(k_scratch) & 127u) != 0) return fail(ctx, PRECC_ERR_MISALIGNED, "key scratch not 128-byte aligned");
  PrefillArgs b = a;
  b.rope = nullptr; b.max_pos = 0; b.B_k = nullptr; b.k_scratch = k_scratch; b.k_scratch_blocks = out_blocks;
  const int32_t ok = desc->head_dim == 64 ? prefill_tc_eligible_hd64(ctx, b, 0, rv) : prefill_tc_eligible_hd128(ctx, b, 0, rv);
  if (ok < 0) return ok;
  if (ok == 0) return run();
  RopeExpandParams x;
  const size_t kvw = (size_t)desc->n_kv_heads * desc->head_dim;
  x.k_base = (const __nv_bfloat16*)cache->k_base;
  x.lr_k = (const __nv_bfloat16*)cache->lr_k + (size_t)agent * cache->n_blocks * PRECC_PAGE * desc->rank_k;
  x.B_k = (const __nv_bfloat16*)B_k + (size_t)agent * desc->rank_k * kvw;
  x.rope = reinterpret_cast<const float4*>(rope->table);
  x.block_table = block_table; x.scratch = (__nv_bfloat16*)k_scratch; x.status = ctx->status;
  x.n_blocks = cache->n_blocks; x.first_block = first_block; x.n_tokens = ctx_len + S;
  x.n_kv = desc->n_kv_heads; x.hd = desc->head_dim; x.rk = desc->rank_k; x.max_pos = rope->max_pos; x.s_k = desc->lora_scale_k;
  x.n_out_blocks = (int)out_blocks;
  const int n_tasks = desc->n_kv_heads * (desc->head_dim / 32);
  auto launch = [&](auto kern, size_t xs, int group_tasks) -> int32_t {
    PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, (int)xs));
    const int groups = (n_tasks + group_tasks - 1) / group_tasks;
    long long gx = 2ll * ctx->sm_count / groups;          // two resident blocks per SM: each walks its share of the cache blocks
    if (gx < 1) gx = 1;
    if (gx > out_blocks) gx = out_blocks;
    kern<<<dim3((unsigned)gx, (unsigned)groups), RX_THREADS, xs, (cudaStream_t)stream>>>(x);
    PRECC_CUDA(ctx, cudaGetLastError());
    return PRECC_OK;
  };
  int32_t xrc;
  if (desc->rank_k <= 16) xrc = launch(rope_expand_keys_kernel<1>, rope_expand_smem_bytes<1>(), RxCfg<1>::GROUP_TASKS);
  else if (desc->rank_k == 32) xrc = launch(rope_expand_keys_kernel<2>, rope_expand_smem_bytes<2>(), RxCfg<2>::GROUP_TASKS);
  else xrc = launch(rope_expand_keys_kernel<4>, rope_expand_smem_bytes<4>(), RxCfg<4>::GROUP_TASKS);
  if (xrc) return xrc;
  return desc->head_dim == 64 ? prefill_run_hd64(ctx, b, 0, rv) : prefill_run_hd128(ctx, b, 0, rv);
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

size_t precc_prefill_ws_bytes(const precc_ctx* ctx, const precc_layer_desc* desc, int32_t S) {
  if (!ctx || !desc || S <= 0 || desc->n_kv_heads <= 0 || desc->n_q_heads < desc->n_kv_heads || desc->head_dim <= 0) return 0;
  const int G = desc->n_q_heads / desc->n_kv_heads;
  if (G > 128) return 0;
  const int tok_per_tile = 128 / G;
  const long long tiles = (long long)((S + tok_per_tile - 1) / tok_per_tile) * desc->n_kv_heads;
  if (tiles * 2 <= ctx->sm_count || tiles > (ctx->sm_count - tiles) * 14) return 0;   // no helper blocks for this turn length (at most 14 tiles per helper)
  const size_t row = (size_t)((desc->head_dim + desc->rank_v + 15) / 16 * 16 + 4);
  const size_t rec = (128 * row + 256) * 4;                                    // one partial: O' rows | m | l
  return ((size_t)tiles * 4 + 255) / 256 * 256 + (size_t)(tiles + ctx->sm_count) * rec;
}

int32_t precc_lr_attend_prefill_ws(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S, int32_t agent,
                                   int32_t ctx_len, const int32_t* block_table, int32_t table_stride, int32_t first_block,
                                   const void* B_k, const void* B_v, const precc_cache* cache, void* out, void* ws,
                                   size_t ws_bytes, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  return prefill_entry(ctx, desc, q, S, agent, ctx_len, block_table, table_stride, first_block, B_k, B_v, nullptr, cache, out, stream,
                       nullptr, 0, ws, ws_bytes);
}

size_t precc_prefill_rope_scratch_bytes(const precc_layer_desc* desc, int32_t ctx_len, int32_t S) {
  if (!desc || ctx_len < 0 || S < 0 || desc->n_kv_heads <= 0 || desc->head_dim <= 0) return 0;
  const long long blocks = ((long long)ctx_len + S + PRECC_PAGE - 1) / PRECC_PAGE;
  const long long stage = 128 / PRECC_PAGE;
  return (size_t)((blocks + stage - 1) / stage * stage) * desc->n_kv_heads * PRECC_PAGE * desc->head_dim * 2;
}

int32_t precc_lr_attend_prefill_rope_scratch(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S, int32_t agent,
                                             int32_t ctx_len, const int32_t* block_table, int32_t table_stride, int32_t first_block,
                                             const void* B_k, const void* B_v, const precc_rope* rope, const precc_cache* cache,
                                             void* out, void* key_scratch, size_t key_scratch_bytes, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!rope) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope is null");
  if (!key_scratch) return fail(ctx, PRECC_ERR_INVALID_ARG, "key scratch is null");
  return prefill_entry(ctx, desc, q, S, agent, ctx_len, block_table, table_stride, first_block, B_k, B_v, rope, cache, out, stream,
                       key_scratch, key_scratch_bytes);
}

}  // extern "C"
