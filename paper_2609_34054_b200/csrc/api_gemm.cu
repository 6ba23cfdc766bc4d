// libprecc: the projection entry points (LR precompute, base re-projection, fused turn projection and
// their rotary forms) and the choice among the three projection kernels.
#include "api_internal.h"
#include "gemm_tc.cuh"
#include "gemm_pair.cuh"
#include "proj_small.cuh"

using namespace precc;

namespace {

// Column tile width.  A block's time per 64-deep k-block hardly depends on the width (measured 0.52 us per k-block
// at 256 columns, 0.45 at 128, 0.42 at 64 and still 0.40 at 16: about 0.40 us + 0.47 ns per column), so a launch
// costs about rounds x that, rounds = ceil(tiles / SMs): the widest tile that does not add a round wins
// (2048 rows x 2304 columns: 144 tiles of 256 in one round, 35 us, against 288 tiles of 128 in two, 55 us), and a
// width that divides the columns evenly beats one whose last tile is half empty (8192 x 1152: 384 tiles of 192
// against 320 of 256, three rounds either way, the narrower ones cheaper).
int pick_bn(int n_out, int m_tiles, int sm_count) {
  if (n_out <= 256) return (n_out + 15) / 16 * 16;
  const int cands[5] = {256, 192, 128, 96, 64};
  int best = 256;
  double best_cost = 1e30;
  for (int i = 0; i < 5; ++i) {
    const long long tiles = (long long)m_tiles * ((n_out + cands[i] - 1) / cands[i]);
    const double cost = (double)((tiles + sm_count - 1) / sm_count) * (0.40 + 0.00047 * cands[i]);
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

int ilog2(int v) { int s = 0; while ((1 << s) < v) ++s; return s; }

int32_t launch_gemm(precc_ctx* ctx, const void* X, int M, int K, const void* Wt, int n_out, GemmParams gp, cudaStream_t stream) {
  gp.hd_shift = ilog2(gp.hd); gp.rk_shift = ilog2(gp.rank_k > 0 ? gp.rank_k : 1); gp.rv_shift = ilog2(gp.rank_v > 0 ? gp.rank_v : 1);
  // Up to 40 rows the weight-streaming few-row kernel is the fastest (fused C3 projection: 5.8 us at 16 rows, 7.4 at
  // 32, 12.7 at 40); from there to about a thousand rows the split-K kernels (12.3 .. 23 us; the few-row kernel needs
  // 12.8 us at 41 rows and 13.7 at 64, the one-block-per-tile GEMM 27 .. 30 us throughout); the few-row kernel still
  // takes 41..64 rows when the split does not apply (rotary epilogue, short K).
  if (M <= 40 && !ctx->force_tiled_gemm) {
    const int32_t rc = launch_small(ctx, X, M, K, Wt, n_out, gp, stream);
    if (rc >= 0) return rc;
  }
  const int m_tiles = (M + GEMM_BM - 1) / GEMM_BM;
  // A few row tiles (the tokens of a short turn): the K extent of every tile is split over a cluster.  The split
  // depends on M and K alone, so a column's summation order is the same whichever entry point produced it.
  if (m_tiles <= 16 && !gp.rope && !ctx->no_gemm_splitk) {
    const int nkb = K / GEMM_BK;
    // planned for the width of the FUSED projection of this layer, whatever this call projects, so that the base-only,
    // LR-only and fused calls of one M take the same decision (and with it the same summation order)
    const int n_fused = 2 * gp.n_kv * gp.hd + gp.n_agents * (gp.rank_k + gp.rank_v);
    // 256-column tiles, one block per SM (a kernel that allocates tensor memory is given one block per SM)
    const int bn = n_out >= 256 ? 256 : (n_out + 15) / 16 * 16;
    const int stage_bytes = GEMM_A_BYTES + 256 * GEMM_BK * 2;
    constexpr int SK_STAGES = 4;                          // ring depth of the split-K kernel
    const int ring_max = SK_STAGES * stage_bytes;
    const long long clusters = (long long)m_tiles * ((n_fused + 255) / 256);
    // the finest split whose clusters are all resident at once (a second wave would cost more than the split gains);
    // cluster sizes need not be powers of two: 18 clusters fit as 6-block clusters, 36 as 3-block clusters
    bool plan_direct = false, plan_push = false;
    int ks = (ctx->gemm_ks_max >= 2 && ctx->gemm_ks_max < GEMM_MAX_KS) ? ctx->gemm_ks_max : GEMM_MAX_KS, smem_plan = 0;
    const int push_max = (ctx->gemm_push_max >= 0 && ctx->gemm_push_max < GEMM_PUSH_MAX_KS) ? ctx->gemm_push_max : GEMM_PUSH_MAX_KS;
    // Clusters of 2 .. 4 blocks merge by bulk sends (proj_gemm_splitk_push_kernel), larger ones by pulling over
    // distributed shared memory (their slices do not fit twice beside each other) or, for up to 64 rows, by direct
    // sends.  Fused Llama-3-8B projection, graph replay over rotating weights: 384 / 512 / 640 rows (clusters of
    // 4 / 4 / 3) 16.4 / 18.4 / 19.2 us against 19.3 / 22.1 / 22.5 us with the pulling merge; 768 / 896 / 1024 rows
    // (clusters of 2) 22.4 / 22.6 / 23.2 us against 29.2 / 30.1 / 30.3 us on the one-block-per-tile kernel (a two-way
    // split did not pay for a pulling merge).
    const int ks_min = ctx->gemm_ks_min;
    for (; ks >= ks_min; --ks) {
      const bool bulk = ks <= push_max && ctx->gemm_direct < 2;       // whole slices by bulk copy
      // pieces straight from registers: pays only while few rows exist (fused Llama-3-8B projection, clusters of 8:
      // 11.7 against 12.2 us at 41 rows, 12.6 against 13.0 at 64, but 16.5 against 15.6 at 128 and 21.8 against 17.0 at 256)
      const bool direct = !bulk && (ctx->gemm_direct >= 2 || (ctx->gemm_direct == 1 && M <= 64));
      const bool push = bulk || direct;
      if (nkb / ks < (ks <= GEMM_PUSH_MAX_KS ? 4 : 2)) continue;       // a coarse split of a short K is not worth a cluster
      const int cw = ((256 + ks - 1) / ks + 7) / 8 * 8;          // planned for the widest tile, whatever this call's width
      const int slice = GEMM_BM * (cw + 4) * 4;
      const int dump = bulk ? 2 * (ks - 1) * slice : (direct ? (ks - 1) * slice : ks * slice);
      smem_plan = (((ring_max > dump ? ring_max : dump) + 1023) & ~1023) + (2 * SK_STAGES + 8) * 8;
      if (smem_plan > ctx->max_smem_optin) continue;
      static int max_clusters_dev[kMaxDevices][2][GEMM_MAX_KS + 1] = {{{0}}};   // 0 = unknown, else max active clusters + 1
      std::lock_guard<std::recursive_mutex> lk(lazy_mu());
      int& cached = max_clusters_dev[ctx->device % kMaxDevices][push ? 1 : 0][ks];
      plan_direct = direct; plan_push = push;
      if (cached == 0) {
        int n = 0;
        auto kern = push ? proj_gemm_splitk_push_kernel : proj_gemm_splitk_kernel;
        if (raise_smem_limit(ctx, kern, smem_plan) == cudaSuccess) {
          cudaLaunchConfig_t qc = {};
          qc.gridDim = dim3(ks, ctx->sm_count, 1); qc.blockDim = dim3(GEMM_THREADS); qc.dynamicSmemBytes = smem_plan;
          cudaLaunchAttribute qa[1];
          qa[0].id = cudaLaunchAttributeClusterDimension;
          qa[0].val.clusterDim.x = ks; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
          qc.attrs = qa; qc.numAttrs = 1;
          if (cudaOccupancyMaxActiveClusters(&n, kern, &qc) != cudaSuccess) { cudaGetLastError(); n = 0; }
        } else {
          cudaGetLastError();
        }
        cached = n + 1;
      }
      if (cached - 1 >= clusters) break;
    }
    if (ks >= ks_min) {
      const int n_tiles = (n_out + bn - 1) / bn;
      int stages = SK_STAGES;
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
      auto kern = plan_push ? proj_gemm_splitk_push_kernel : proj_gemm_splitk_kernel;
      gp.direct_send = plan_direct ? 1 : 0;
      PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, smem_plan));
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(ks, n_tiles, m_tiles);
      cfg.blockDim = dim3(GEMM_THREADS);
      cfg.dynamicSmemBytes = smem_plan;
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = ks; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, kern, map_x, map_w, gp));
      return PRECC_OK;
    }
  }
  if (M <= PS_MAX_M && !ctx->force_tiled_gemm) {
    const int32_t rc = launch_small(ctx, X, M, K, Wt, n_out, gp, stream);
    if (rc >= 0) return rc;
  }
  // Many rows: two SMs per 256 x 256 tile (each stages half of the weight tile), see gemm_pair.cuh.
  if (ctx->gemm_pair && M >= 2 * GEMM_PAIR_BM) {
    const int bn2 = n_out >= 256 ? 256 : (n_out + 15) / 16 * 16;
    if (!(gp.rope && bn2 % gp.hd != 0)) {
      const int stage2 = GEMM_A_BYTES + (bn2 / 2) * GEMM_BK * 2;
      int st2 = (ctx->max_smem_optin - 4096) / stage2;
      if (st2 > 8) st2 = 8;
      if (st2 > K / GEMM_BK) st2 = K / GEMM_BK;
      if (ctx->gemm_stage_cap > 0 && st2 > ctx->gemm_stage_cap) st2 = ctx->gemm_stage_cap;
      if (st2 >= 2) {
        int tc2 = 32;
        while (tc2 < 2 * bn2) tc2 <<= 1;
        const size_t smem2 = (size_t)st2 * stage2 + (2 * st2 + 6) * 8 + 1024;
        CUtensorMap map_x2, map_w2;
        int32_t rc2 = make_map(ctx, &map_x2, X, M, K, GEMM_BM);
        if (rc2) return rc2;
        rc2 = make_map_w(ctx, &map_w2, Wt, n_out, K, bn2 / 2);
        if (rc2) return rc2;
        gp.M = M; gp.N_out = n_out; gp.K = K; gp.BN = bn2; gp.stages = st2; gp.tmem_cols = tc2;
        gp.spread_rows = 1;
        gp.status = ctx->status;
        gp.trace = (ctx->trace && ctx->trace_blocks >= 128) ? ctx->trace : nullptr;     // used by PRECC_GEMM_TRACE builds only
        PRECC_CUDA(ctx, raise_smem_limit(ctx, proj_gemm_pair_kernel, (int)smem2));
        const long long tiles2 = (long long)((M + GEMM_PAIR_BM - 1) / GEMM_PAIR_BM) * ((n_out + bn2 - 1) / bn2);
        const int pairs = (int)(tiles2 < ctx->sm_count / 2 ? tiles2 : ctx->sm_count / 2);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * pairs);
        cfg.blockDim = dim3(GEMM_THREADS);
        cfg.dynamicSmemBytes = smem2;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        PRECC_CUDA(ctx, cudaLaunchKernelEx(&cfg, proj_gemm_pair_kernel, map_x2, map_w2, gp));
        return PRECC_OK;
      }
    }
  }
  int bn = pick_bn(n_out, m_tiles, ctx->sm_count);
  if (gp.rope && bn % gp.hd != 0) bn = 256;          // a head's two halves must sit in one tile (head_dim 64 or 128 divides 256)
  const int n_tiles = (n_out + bn - 1) / bn;
  const int stage_bytes = GEMM_A_BYTES + bn * GEMM_BK * 2;
  int stages = (ctx->max_smem_optin - 4096) / stage_bytes;
  if (stages > 8) stages = 8;
  if (stages > K / GEMM_BK) stages = K / GEMM_BK;
  if (ctx->gemm_stage_cap > 0 && stages > ctx->gemm_stage_cap) stages = ctx->gemm_stage_cap;
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
  gp.trace = (ctx->trace && ctx->trace_blocks >= 128) ? ctx->trace : nullptr;     // used by PRECC_GEMM_TRACE builds only
  PRECC_CUDA(ctx, raise_smem_limit(ctx, proj_gemm_kernel, (int)smem));
  const int total_tiles = m_tiles * n_tiles;
  proj_gemm_kernel<<<dim3(total_tiles < ctx->sm_count ? total_tiles : ctx->sm_count), GEMM_THREADS, smem, stream>>>(map_x, map_w, gp);
  PRECC_CUDA(ctx, cudaGetLastError());
  return PRECC_OK;
}

}  // namespace

extern "C" {

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
                          const precc_cache* cache, void* stream, const uint64_t* row_masks = nullptr,
                          const int32_t* lr_copy_slots = nullptr) {
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
  gp.lr_copy_slots = lr_copy_slots;
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
                                const int32_t* slot_mapping, const uint64_t* row_agent_masks, const int32_t* lr_copy_slots,
                                const precc_cache* cache, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!slot_mapping || !row_agent_masks) return fail(ctx, PRECC_ERR_INVALID_ARG, "slot_mapping / row_agent_masks is null");
  if (reinterpret_cast<uintptr_t>(row_agent_masks) & 7u) return fail(ctx, PRECC_ERR_MISALIGNED, "row_agent_masks not 8-byte aligned");
  return turn_entry(ctx, desc, H, M, WA_packed, slot_mapping, 0, 0, nullptr, cache, stream, row_agent_masks, lr_copy_slots);
}

int32_t precc_turn_project_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M, const void* WA_packed,
                                const int32_t* slot_mapping, int64_t start_slot, uint64_t agent_mask, const precc_rope* rope,
                                const precc_cache* cache, void* stream) {
  if (!ctx) return PRECC_ERR_INVALID_ARG;
  if (!rope) return fail(ctx, PRECC_ERR_INVALID_ARG, "rope is null");
  return turn_entry(ctx, desc, H, M, WA_packed, slot_mapping, start_slot, agent_mask, rope, cache, stream);
}

}  // extern "C"
