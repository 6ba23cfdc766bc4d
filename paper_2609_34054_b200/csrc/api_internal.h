// Internals shared by the translation units of libprecc (host side): the context, error plumbing,
// argument checks, tensor-map helpers and the per-head-dimension dispatchers that let the attention
// kernels compile in separate units.
#pragma once
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
#include "common.cuh"

struct precc_ctx {
  int device = 0;
  int sm_count = 0;
  int max_smem_optin = 0;
  uint32_t* status = nullptr;          // two device words: [0] status bits, [1] limit of the bounded waits (x 1024 cycles)
  unsigned long long* trace = nullptr; // optional caller-owned trace buffer
  size_t trace_blocks = 0;
  bool force_simple_prefill = false;   // PRECC_PREFILL=simple in the environment
  int gemm_stage_cap = 0;              // PRECC_GEMM_STAGES=n in the environment: ring depth of the tiled GEMMs at most n (experiments)
  bool gemm_pair = false;              // PRECC_GEMM=pair in the environment: two SMs per tile for projections of many rows
  bool force_tiled_gemm = false;       // PRECC_GEMM=tiled in the environment: never take the few-row kernel
  int gemm_ks_max = 0;                 // PRECC_GEMM_KS_MAX=n: finest K split (0 = the largest the kernels support)
  int gemm_push_max = -1;              // PRECC_GEMM_PUSH_MAX=n: merge by bulk sends up to this split (-1 = the kernels' limit, 0 = never)
  int gemm_direct = 1;                 // PRECC_GEMM_DIRECT=n: split-K merge by direct sends - 0 never, 1 finer splits of up to 64 rows, 2 every split
  int gemm_ks_min = 2;                 // PRECC_GEMM_KS_MIN=n in the environment: coarsest K split of short-turn projections (experiments)
  bool no_gemm_splitk = false;         // PRECC_GEMM_SPLITK=0 in the environment: short turns stay on the one-block-per-tile GEMM
  bool force_ticket_decode = false;    // PRECC_DECODE=ticket in the environment: never use the cluster decode kernel
  bool deep_clusters = true;           // PRECC_DEEP=0 in the environment: never use the one-block-per-SM deep-ring clusters
  bool deep_always = false;            // PRECC_DEEP=2: take them wherever they fit, also where they leave many SMs without a block
  int decode_pre_stages = 0;           // PRECC_DECODE_PRE=n in the environment: ring slots filled before the dependency wait (0 = all)
  int decode_stage_cap = 0;            // PRECC_DECODE_STAGES=n in the environment: at most n ring slots per warp in the cluster schedule (0 = planner's choice)
  int decode_cluster_policy = 0;       // PRECC_DECODE_POLICY=n in the environment: cluster scheduling policy of the decode clusters - 0 the driver's default, 1 spread, 2 load balancing
  int decode_cluster_cap = 0;          // PRECC_DECODE_CLUSTER=n in the environment: at most n blocks per decode cluster (0 = planner's choice)
  bool prefill_forward = false;        // PRECC_PREFILL_ORDER=forward: row tiles in ascending order (default: longest causal reach first)
  bool no_prefill_split = false;       // PRECC_PREFILL_SPLIT=0 in the environment: never split a turn's context over a cluster
  bool no_prefill_vhalf = false;       // PRECC_PREFILL_VHALF=0 in the environment: the value ring of the tcgen05 prefill kernel always holds whole steps
  bool no_prefill_helpers = false;     // PRECC_PREFILL_HELPERS=0 in the environment: prefill with a workspace never uses helper blocks
  int prefill_helper_p = 0;            // PRECC_PREFILL_HELPER_P=n in the environment: the tiles' own blocks stop after n steps (experiments; 0 = planner's choice)
  int prefill_helper_min_steps = 48;   // PRECC_PREFILL_HELPER_MIN=n in the environment: shortest context (128-token steps) that gets helper blocks
  char err[512] = {0};
  CUresult (*encode_tiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                           const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                           CUtensorMapL2promotion, CUtensorMapFloatOOBfill) = nullptr;
};

namespace precc {

constexpr int kMaxDevices = 64;
constexpr uint32_t kDefaultWaitLimit = 2000000000u >> 10;   // about a second of SM clock, in units of 1024 cycles

int32_t fail(precc_ctx* ctx, int32_t code, const char* fmt, ...);

#define PRECC_CUDA(ctx, expr)                                                                   \
  do {                                                                                          \
    cudaError_t e__ = (expr);                                                                   \
    if (e__ != cudaSuccess) return fail(ctx, PRECC_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)


// Dynamic shared-memory limit of a kernel on the context's device: only ever raised (a kernel serves
// several configurations; lowering the limit for a small one would make a later large launch fail), and
// set under a lock so that contexts on several host threads cannot interleave a set and a launch badly.
cudaError_t raise_smem_limit_raw(precc_ctx* ctx, const void* fn, int bytes);
template <typename K>
cudaError_t raise_smem_limit(precc_ctx* ctx, K kern, int bytes) {
  return raise_smem_limit_raw(ctx, reinterpret_cast<const void*>(kern), bytes);
}
// Guards the per-device answers that are looked up once and kept for the life of the process (occupancy of
// a cluster shape, kernel attributes, the address of the built-in scratch array): contexts on different
// host threads may ask for them at the same time.
std::recursive_mutex& lazy_mu();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool rank_ok(int r) { return r == 8 || r == 16 || r == 32 || r == 64; }
int32_t check_desc(precc_ctx* ctx, const precc_layer_desc* d);
int32_t check_cache(precc_ctx* ctx, const precc_layer_desc* d, const precc_cache* c, bool need_base, bool need_lr);
float softmax_scale_log2(const precc_layer_desc* d);

int32_t make_map(precc_ctx* ctx, CUtensorMap* map, const void* base, int rows, int cols, int box_rows);
int32_t make_map_w(precc_ctx* ctx, CUtensorMap* map, const void* base, int rows, int K, int box_rows);
int32_t make_map2(precc_ctx* ctx, CUtensorMap* map, const void* base, long long rows, int cols, int box_rows, int box_cols);
int32_t make_map_cache4(precc_ctx* ctx, CUtensorMap* map, const void* base, long long n_blocks, int n_kv, int hd, int box_blocks);

// F<HD, RK, RV>::run(ctx, args...) for the rank pair (rk, rv) of one head dimension.
template <template <int, int, int> class F, int HD, typename... Args>
int32_t dispatch_ranks(precc_ctx* ctx, int rk, int rv, Args&&... args) {
#define PRECC_CASE(RK, RV) \
  if (rk == RK && rv == RV) return F<HD, RK, RV>::run(ctx, args...);
  PRECC_CASE(0, 0) PRECC_CASE(0, 8) PRECC_CASE(0, 16) PRECC_CASE(0, 32) PRECC_CASE(0, 64)
  PRECC_CASE(8, 8) PRECC_CASE(16, 16) PRECC_CASE(32, 32) PRECC_CASE(64, 64)
#undef PRECC_CASE
  return fail(ctx, PRECC_ERR_UNSUPPORTED, "no kernel for head_dim %d ranks (%d,%d)", HD, rk, rv);
}

struct DecodeArgs {
  const precc_layer_desc* d; const void* q; int B; const int32_t* agent_id; const int32_t* ctx_len;
  const int32_t* block_table; int table_stride; const int32_t* first_block; int max_ctx;
  const void* B_k; const void* B_v; const precc_cache* cache; void* out; void* ws; size_t ws_bytes; cudaStream_t stream;
  const float* rope = nullptr; int max_pos = 0;      // rotary variant when rope != null
  float* raw = nullptr;                              // partial-output mode: records instead of `out`
  bool clear_counters = false;                       // zero the arrival counters on the stream before a launch that uses them
};

struct PrefillArgs {
  const precc_layer_desc* d; const void* q; int S; int agent; int T; const int32_t* block_table; int first_block;
  const void* B_k; const void* B_v; const precc_cache* cache; void* out; cudaStream_t stream;
  const float* rope = nullptr; int max_pos = 0;      // rotary variant when rope != null
  const void* k_scratch = nullptr;                   // adapted keys of this sequence in logical block order (rotary prefill
  long long k_scratch_blocks = 0;                    // with scratch): the keys come from here, the values from the cache
  void* ws = nullptr; size_t ws_bytes = 0;           // optional workspace of the work-list launch (helper blocks on idle SMs)
};


struct WsQuery { int sm_count, max_smem, B, n_kv, max_ctx; size_t* out; };

// One definition per head dimension, each in its own translation unit (rotary variant when a.rope != null).
int32_t decode_run_hd64(precc_ctx* ctx, const DecodeArgs& a);
int32_t decode_run_hd128(precc_ctx* ctx, const DecodeArgs& a);
int32_t decode_ws_hd64(precc_ctx* ctx, int rk, int rv, const WsQuery& w);
int32_t decode_ws_hd128(precc_ctx* ctx, int rk, int rv, const WsQuery& w);
int32_t prefill_run_hd64(precc_ctx* ctx, const PrefillArgs& a, int rk, int rv);
int32_t prefill_run_hd128(precc_ctx* ctx, const PrefillArgs& a, int rk, int rv);
// 1 when the tensor-memory prefill kernel would take the call, 0 when not, negative on an unsupported rank pair
int32_t prefill_tc_eligible_hd64(precc_ctx* ctx, const PrefillArgs& a, int rk, int rv);
int32_t prefill_tc_eligible_hd128(precc_ctx* ctx, const PrefillArgs& a, int rk, int rv);

}  // namespace precc
