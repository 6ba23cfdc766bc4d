// Host side of new-turn prefill attention: kernel choice (tcgen05 kernel or the mma.sync kernel), tensor maps,
// the cluster split of short turns and the launch.  Included by one translation unit per head dimension.
#pragma once
#include <algorithm>
#include <vector>

#include "api_internal.h"
#include "prefill.cuh"
#include "prefill_tc.cuh"

namespace precc {

template <int HD, int RK, int RV>
struct PrefillRun {
  // ---- work-list launch of the tensor-core kernel: plan and workspace
  struct WorkList { int p = 0, helpers = 0, tiles = 0; };
  static size_t ticket_bytes(int tiles) { return ((size_t)tiles * 4 + 255) / 256 * 256; }
  static size_t worklist_ws_bytes(int tiles, int helpers) {
    return ticket_bytes(tiles) + (size_t)(2 * tiles + helpers) * PrefillTcCfg<HD, RK, RV>::REC_FLOATS * 4;
  }
  // Steps of row tile x; the tail of a tile is what lies beyond the first `p` steps.  Tails are laid end to end, kv
  // head by kv head, and cut into `helpers` equal ranges (the kernel derives the same cuts from p and helpers).
  // The cost of a plan, in steps: the longer of a tile's own block (p + its record and possibly the merge) and a
  // helper (its range + a drain and refill per piece).  Returns p = 0 when the classic launch is as good.
  static WorkList plan_worklist(precc_ctx* ctx, int S, int T, int tok_per_tile, int n_kv) {
    WorkList best;
    if (ctx->no_prefill_helpers) return best;
    const int X = (S + tok_per_tile - 1) / tok_per_tile;
    const long long tiles = (long long)X * n_kv;
    const int H = ctx->sm_count - (int)tiles;
    if (X >= PTC_MAX_XT || tiles * 2 <= ctx->sm_count || tiles > (long long)H * (PTC_MAX_SEG - 2)) return best;
    auto steps_of = [&](int x) { return (int)(((long long)T + std::min(S, (x + 1) * tok_per_tile) + PTC_TOK - 1) / PTC_TOK); };
    const int n_max = steps_of(X - 1);
    if (n_max < ctx->prefill_helper_min_steps) return best;
    // what a record + merge costs a tile's own block, and what a piece costs a helper beyond its steps (query tile,
    // fold, pipeline fill, record), in steps: measured at head_dim 128, rank 32 (1.3 us per step), scaled for shorter steps
    const int f100 = 100 * 160 / (HD + (RK + RV) / 2);
    const int C_OWN = 14 * f100 / 100, C_PIECE = 12 * f100 / 100;
    int best_cost = n_max - std::max(2, n_max / 12);   // a plan must win at least 8 % on paper: with every SM busy a step takes about 4 % longer
    for (int p = n_max - 1; p >= std::max(8, n_max / 2); --p) {
      if (ctx->prefill_helper_p > 0 && p != ctx->prefill_helper_p) continue;
      long long tail_sum = 0;
      for (int x = 0; x < X; ++x) tail_sum += std::max(0, steps_of(x) - p);
      const long long total = tail_sum * n_kv;
      const long long per = std::max(1ll, (total + H - 1) / H);
      if (p + C_OWN >= best_cost && ctx->prefill_helper_p <= 0) continue;
      // walk the tails in the kernel's order: pieces per helper and pieces per tile
      int max_seg = 0, max_src = 0;
      long long pos = 0;
      for (int g = 0; g < n_kv; ++g)
        for (int x = 0; x < X; ++x) {
          const int tl = std::max(0, steps_of(x) - p);
          if (tl == 0) continue;
          const long long hf = pos / per, hl = (pos + tl - 1) / per;
          max_src = std::max(max_src, (int)(2 + hl - hf));
          pos += tl;
        }
      {
        // pieces of helper h = tiles whose tail range meets [h per, (h+1) per)
        std::vector<int> cnt(H, 0);
        pos = 0;
        for (int g = 0; g < n_kv; ++g)
          for (int x = 0; x < X; ++x) {
            const int tl = std::max(0, steps_of(x) - p);
            if (tl == 0) continue;
            for (long long h = pos / per; h <= (pos + tl - 1) / per && h < H; ++h) ++cnt[(size_t)h];
            pos += tl;
          }
        for (int h = 0; h < H; ++h) max_seg = std::max(max_seg, cnt[(size_t)h]);
      }
      if (max_seg > PTC_MAX_SEG || max_src > PTC_MAX_SRC) continue;
      const int cost = (int)std::max<long long>(p + C_OWN, per + (long long)C_PIECE * max_seg);
      if (cost < best_cost || ctx->prefill_helper_p > 0) { best_cost = cost; best.p = p; best.helpers = H; best.tiles = (int)tiles; }
    }
    return best;
  }
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
    // room for one value stage but not for two (head_dim 128 with rank 64): a ring of three 64-token half stages
    // lets the next step's values start loading while the current step's are still being read
    bool v_half = false;
    if constexpr (C::V_HALF_CAPABLE) {
      if (vs == 1 && !ctx->no_prefill_vhalf && C::smem_bytes(ks, 3, true) <= ctx->max_smem_optin) { v_half = true; vs = 3; }
    }
    const int smem = C::smem_bytes(ks, vs, v_half);
    const size_t kvw = (size_t)d->n_kv_heads * HD;
    const long long kv_rows = (long long)a.cache->n_blocks * d->n_kv_heads * PAGE;
    const long long lr_rows = (long long)a.cache->n_blocks * PAGE;
    CUtensorMap mk, mv, mlk, mlv;
    // without a block table the pages of a 128-token stage are consecutive: whole-stage boxes (one TMA
    // instruction per 64-column slab instead of one per page)
    const bool contig = a.block_table == nullptr;
    const int box_rows = contig ? PTC_TOK : PAGE;
    const int v_box_blocks = (v_half ? PTC_TOK / 2 : PTC_TOK) / PAGE, v_box_rows = contig ? v_box_blocks * PAGE : PAGE;
    int32_t rc = a.k_scratch ? make_map_cache4(ctx, &mk, a.k_scratch, a.k_scratch_blocks, d->n_kv_heads, HD, PTC_TOK / PAGE)
                 : contig    ? make_map_cache4(ctx, &mk, a.cache->k_base, a.cache->n_blocks, d->n_kv_heads, HD, PTC_TOK / PAGE)
                             : make_map2(ctx, &mk, a.cache->k_base, kv_rows, HD, PAGE, 64);
    if (rc) return rc;
    rc = contig ? make_map_cache4(ctx, &mv, a.cache->v_base, a.cache->n_blocks, d->n_kv_heads, HD, v_box_blocks)
                : make_map2(ctx, &mv, a.cache->v_base, kv_rows, HD, PAGE, 64);
    if (rc) return rc;
    mlk = mk; mlv = mv;     // placeholders when a rank is zero (never dereferenced)
    if (RK) { rc = make_map2(ctx, &mlk, (const __nv_bfloat16*)a.cache->lr_k + (size_t)a.agent * lr_rows * RK, lr_rows, RK, box_rows, C::RKP); if (rc) return rc; }
    if (RV) { rc = make_map2(ctx, &mlv, (const __nv_bfloat16*)a.cache->lr_v + (size_t)a.agent * lr_rows * RV, lr_rows, RV, v_box_rows, 64); if (rc) return rc; }
    PrefillTcParams p;
    p.q = (const __nv_bfloat16*)a.q; p.out = (__nv_bfloat16*)a.out; p.block_table = a.block_table;
    p.B_k = RK ? (const __nv_bfloat16*)a.B_k + (size_t)a.agent * RK * kvw : nullptr;
    p.B_v = RV ? (const __nv_bfloat16*)a.B_v + (size_t)a.agent * RV * kvw : nullptr;
    p.status = ctx->status; p.n_blocks = a.cache->n_blocks;
    p.S = a.S; p.T = a.T; p.first_block = a.first_block; p.contig = contig ? 1 : 0; p.k_logical = a.k_scratch ? 1 : 0;
    p.longest_first = ctx->prefill_forward ? 0 : 1;
    p.n_q = d->n_q_heads; p.n_kv = d->n_kv_heads; p.group = G; p.tok_per_tile = PTC_TOK / G; p.k_stages = ks; p.v_stages = vs; p.v_half = v_half ? 1 : 0;
    p.scale_log2 = softmax_scale_log2(d); p.s_k = d->lora_scale_k; p.s_v = d->lora_scale_v;
    p.trace = (ctx->trace && ctx->trace_blocks >= 32) ? ctx->trace : nullptr;
    // four instantiations at most: classic / work list, whole-step / half-step value ring (the latter only where it applies)
    using KernT = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, PrefillTcParams);
    KernT kern = lr_attend_prefill_tc_kernel<HD, RK, RV, false, false>;
    KernT kern_wl = lr_attend_prefill_tc_kernel<HD, RK, RV, true, false>;
    if constexpr (C::V_HALF_CAPABLE) {
      if (v_half) { kern = lr_attend_prefill_tc_kernel<HD, RK, RV, false, true>; kern_wl = lr_attend_prefill_tc_kernel<HD, RK, RV, true, true>; }
    }
    PRECC_CUDA(ctx, raise_smem_limit(ctx, kern, smem));
    const int row_tiles = (a.S + p.tok_per_tile - 1) / p.tok_per_tile;
    // Short turn over a long context: too few (row tile, kv head) blocks to fill the machine, so the
    // context of each is split over a cluster of up to 8 blocks whose partial results merge over DSMEM.
    int ns = 1;
    const long long base_blocks = (long long)row_tiles * d->n_kv_heads;
    const int steps = (a.T + a.S + PTC_TOK - 1) / PTC_TOK;
    if (!ctx->no_prefill_split && C::SPLIT_BYTES <= C::Q_BYTES + C::QX_BYTES + ks * C::KSTAGE + vs * (v_half ? C::VSTAGE / 2 : C::VSTAGE)) {
      ns = (int)(ctx->sm_count / base_blocks);          // as many as keep the grid within one block per SM
      if (ns > 8) ns = 8;
      if (ns > steps / 8) ns = steps / 8;               // at least eight steps per block
      if (ns < 1) ns = 1;
      // every cluster must be resident at once (one block per SM, and a cluster lives inside one GPC): ask
      // the occupancy calculator once per cluster size, and shrink the clusters until the grid fits in one wave
      static int max_clusters_dev[kMaxDevices][9] = {{0}};   // 0 = unknown, else max active clusters + 1
      std::lock_guard<std::recursive_mutex> lk(lazy_mu());
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
    p.helper_p = 0; p.n_helpers = 0; p.row_tiles = row_tiles; p.ws_rec = nullptr; p.ws_ticket = nullptr;
    // One wave that leaves SMs without a block (a 512-token turn of 8 kv heads is 128 blocks on 148 SMs): with a
    // workspace the blocks stop `helper_p` steps into their tile and helper blocks on the idle SMs share the tails.
#ifdef PRECC_PF_TRACE
    const bool wl_ok = !p.trace || ctx->trace_blocks >= 2048;   // room for every block's piece stamps
#else
    const bool wl_ok = !p.trace;
#endif
    if (a.ws && ns == 1 && wl_ok) {
      const WorkList wl = plan_worklist(ctx, a.S, a.T, p.tok_per_tile, d->n_kv_heads);
      if (wl.p > 0 && a.ws_bytes >= worklist_ws_bytes(wl.tiles, wl.helpers)) {
        p.helper_p = wl.p; p.n_helpers = wl.helpers; p.longest_first = 0;
        p.ws_ticket = reinterpret_cast<unsigned int*>(a.ws);
        p.ws_rec = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(a.ws) + ticket_bytes(wl.tiles));
        PRECC_CUDA(ctx, cudaMemsetAsync(a.ws, 0, ticket_bytes(wl.tiles), a.stream));
        PRECC_CUDA(ctx, raise_smem_limit(ctx, kern_wl, smem));
        cudaLaunchConfig_t wc = {};
        wc.gridDim = dim3(wl.tiles + wl.helpers); wc.blockDim = dim3(PTC_THREADS); wc.dynamicSmemBytes = smem; wc.stream = a.stream;
        PRECC_CUDA(ctx, cudaLaunchKernelEx(&wc, kern_wl, mk, mv, mlk, mlv, p));
        return PRECC_OK;
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
  // whether the tensor-memory kernel takes this call (shape, cache size, alignment, diagnostic switch)
  static bool tc_eligible(precc_ctx* ctx, const PrefillArgs& a) {
    if constexpr (PrefillTcCfg<HD, RK, RV>::supported) {
      const long long kv_rows = (long long)a.cache->n_blocks * a.d->n_kv_heads * PAGE;
      const bool aligned128 = ((reinterpret_cast<uintptr_t>(a.cache->k_base) | reinterpret_cast<uintptr_t>(a.cache->v_base) |
                                reinterpret_cast<uintptr_t>(a.cache->lr_k) | reinterpret_cast<uintptr_t>(a.cache->lr_v) |
                                reinterpret_cast<uintptr_t>(a.k_scratch)) & 127u) == 0;
      return kv_rows < (1ll << 31) && aligned128 && !ctx->force_simple_prefill;
    }
    return false;
  }
  static int32_t run(precc_ctx* ctx, const PrefillArgs& a) {
    if (tc_eligible(ctx, a)) {
      if constexpr (PrefillTcCfg<HD, RK, RV>::supported) return run_tc(ctx, a);
    }
    if (a.k_scratch) return fail(ctx, PRECC_ERR_UNSUPPORTED, "prefill from a key scratch needs the tensor-memory kernel");
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


template <int HD, int RK, int RV>
struct PrefillEligible {
  static int32_t run(precc_ctx* ctx, const PrefillArgs& a) { return PrefillRun<HD, RK, RV>::tc_eligible(ctx, a) ? 1 : 0; }
};

}  // namespace precc

#define PRECC_DEFINE_PREFILL_UNIT(HD)                                                                         \
  namespace precc {                                                                                           \
  int32_t prefill_tc_eligible_hd##HD(precc_ctx* ctx, const PrefillArgs& a, int rk, int rv) {                  \
    return dispatch_ranks<PrefillEligible, HD>(ctx, rk, rv, a);                                               \
  }                                                                                                           \
  int32_t prefill_run_hd##HD(precc_ctx* ctx, const PrefillArgs& a, int rk, int rv) {                          \
    if (a.rope) return dispatch_ranks<PrefillRunRope, HD>(ctx, rk, rv, a);                                    \
    return dispatch_ranks<PrefillRun, HD>(ctx, rk, rv, a);                                                    \
  }                                                                                                           \
  }
