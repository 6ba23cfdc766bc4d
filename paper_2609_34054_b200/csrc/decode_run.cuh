// Host side of decode attention: the split schedule (cluster kernel or ticket kernel), workspace sizing and
// the launch.  Included by one translation unit per head dimension.
#pragma once
#include "api_internal.h"
#include "decode.cuh"

namespace precc {

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

// Warps of a cluster-schedule block when two blocks share an SM (8 if a two-page ring per warp fits, else 4).
template <int HD, int RK, int RV>
int two_per_sm_warps(int max_smem, int extra) {
  return DecodeCfg<HD, RK, RV>::cluster_smem(8, 2) <= max_smem / 2 - 1024 - extra ? 8 : 4;
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
  int warps = 8, stages = 8;
  while (stages > 2 && C::cluster_smem(8, stages) > budget) --stages;
  if (C::cluster_smem(8, stages) > budget) {
    warps = 4; stages = 8;
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

template <int HD, int RK, int RV, bool ROPE = false>
struct DecodeRunT {
  // The workspace bound below is computed for the plain kernel and serves the rotary one too: the rotary blocks
  // are larger (the B_k slice rides in shared memory), which can only lower the split count - as long as two
  // of them still fit on an SM at the shallowest ring, so that the planner's blocks-per-SM figure is the same.
  static_assert(!ROPE || 2 * (DecodeCfg<HD, RK, RV>::ticket_smem(2) + DecodeCfg<HD, RK, RV>::BK_BYTES + 128 + 1024) <= 232448,
                "rotary ticket blocks must fit two per SM, or the workspace bound of the plain kernel no longer covers them");
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
    std::lock_guard<std::recursive_mutex> lk(lazy_mu());
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
    std::lock_guard<std::recursive_mutex> lk(lazy_mu());
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
    // planner's choice, then the experiment switches of the environment
    auto plan = [&](bool deep) {
      DecodePlan q = plan_cluster<HD, RK, RV>(ctx->sm_count, ctx->max_smem_optin, a.B, d->n_kv_heads, a.max_ctx, extra, deep);
      if (ctx->force_ticket_decode) q.cluster = 0;
      if (q.cluster > 1 && ctx->decode_cluster_cap > 1 && q.cluster > ctx->decode_cluster_cap) {
        const int mt = (a.max_ctx + PAGE - 1) / PAGE;
        q.cluster = ctx->decode_cluster_cap; q.chunk_tiles = (mt + q.cluster - 1) / q.cluster; q.max_splits = q.cluster;
      }
      if (q.cluster > 1 && ctx->decode_stage_cap >= 2 && q.stages > ctx->decode_stage_cap) {
        q.stages = ctx->decode_stage_cap;
        q.smem = DecodeCfg<HD, RK, RV>::cluster_smem(q.warps, q.stages) + extra;
      }
      return q;
    };
    DecodePlan pl = plan(deep_ok);
    auto fits = [&](const DecodePlan& q) { return q.warps == 8 ? cluster_fits<8>(ctx, q, a.B * d->n_kv_heads) : cluster_fits<4>(ctx, q, a.B * d->n_kv_heads); };
    if (pl.cluster && pl.deep) {
      const int max_tiles = (a.max_ctx + PAGE - 1) / PAGE;
      while (pl.cluster > 4 && !fits(pl)) { --pl.cluster; pl.chunk_tiles = (max_tiles + pl.cluster - 1) / pl.cluster; pl.max_splits = pl.cluster; }
      if (pl.cluster <= 4) pl.cluster = 0;
      // One block per SM means at most one cluster of more than half a GPC per GPC: 8 units get 10-block clusters,
      // 80 of 148 SMs.  Where two 8-warp blocks fit on an SM the two-blocks-per-SM layout (16-block clusters, or
      // the ticket kernel for long contexts) reaches more SMs and is faster then (head_dim 64, one request:
      // 8192 tokens 8.0 -> 7.1 us, 131072 tokens 60 -> 49 us); with 4-warp blocks (head_dim 128) the deep rings win.
      if (!ctx->deep_always && pl.cluster * a.B * d->n_kv_heads * 4 < ctx->sm_count * 3 &&
          two_per_sm_warps<HD, RK, RV>(ctx->max_smem_optin, extra) == 8) {
        pl = plan(false);
        if (pl.cluster && !fits(pl)) pl.cluster = 0;
      }
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
    p.chunk_tiles = pl.chunk_tiles; p.max_splits = pl.max_splits; p.stages = pl.stages; p.max_ctx = a.max_ctx;
    p.pre_stages = (ctx->decode_pre_stages >= 1 && ctx->decode_pre_stages < pl.stages) ? ctx->decode_pre_stages : pl.stages;
    p.scale_log2 = softmax_scale_log2(d); p.s_k = d->lora_scale_k; p.s_v = d->lora_scale_v;
    p.rope = reinterpret_cast<const float4*>(a.rope); p.max_pos = a.max_pos;
    p.bk_off = ROPE ? ((pl.smem - extra + 127) / 128) * 128 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.max_splits, d->n_kv_heads, a.B);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[3];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (pl.cluster) {
      cfg.blockDim = dim3(pl.warps * 32);
      attr[1].id = cudaLaunchAttributeClusterDimension;
      attr[1].val.clusterDim.x = pl.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
      cfg.numAttrs = 2;
      if (ctx->decode_cluster_policy) {
        // where the blocks of a cluster go inside their GPC: spread over as many SMs as possible, or packed
        attr[2].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
        attr[2].val.clusterSchedulingPolicyPreference =
            ctx->decode_cluster_policy == 1 ? cudaClusterSchedulingPolicySpread : cudaClusterSchedulingPolicyLoadBalancing;
        cfg.numAttrs = 3;
      }
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
      if (a.clear_counters) PRECC_CUDA(ctx, cudaMemsetAsync(p.tickets, 0, tickets, a.stream));
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


template <int HD, int RK, int RV>
struct DecodeWs {
  static int32_t run(precc_ctx*, const WsQuery& w) {
    *w.out = DecodeRun<HD, RK, RV>::ws_bytes(w.sm_count, w.max_smem, w.B, w.n_kv, w.max_ctx);
    return PRECC_OK;
  }
};

}  // namespace precc

#define PRECC_DEFINE_DECODE_UNIT(HD)                                                                          \
  namespace precc {                                                                                           \
  int32_t decode_run_hd##HD(precc_ctx* ctx, const DecodeArgs& a) {                                            \
    if (a.rope) return dispatch_ranks<DecodeRunRope, HD>(ctx, a.d->rank_k, a.d->rank_v, a);                   \
    return dispatch_ranks<DecodeRun, HD>(ctx, a.d->rank_k, a.d->rank_v, a);                                   \
  }                                                                                                           \
  int32_t decode_ws_hd##HD(precc_ctx* ctx, int rk, int rv, const WsQuery& w) {                                \
    return dispatch_ranks<DecodeWs, HD>(ctx, rk, rv, w);                                                      \
  }                                                                                                           \
  }
