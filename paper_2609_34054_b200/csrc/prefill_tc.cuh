// LR-reconstructed attention for the new tokens of a turn on the 5th-generation tensor cores.
//
// One thread block = up to 128 query rows of one kv head (row = new token i * G + head-in-group) against
// the whole visible context, 128 tokens per step:
//   S  = Q K_base^T + Q~ L_K^T                 tcgen05.mma, A/B from shared memory, S in TMEM (2 buffers)
//   P  = exp2(S*scale - m)                     8 softmax warps, two threads per TMEM lane (= query row);
//                                              packed bf16 in its own 64 TMEM columns
//   O' += P [V_base | L_V | 1]                  tcgen05.mma with A = P from TMEM; O' in TMEM holds the numerator
//                                              (hd columns), U = P L_V (r_v columns) and, through a column of
//                                              ones written into the zero-padded L_V slab, the denominator
// and finally out = (O + s_v U B_v) / l on the CUDA cores.  The key-side fold Q~ = s_k Q B_k^T is one
// small MMA chain per block before the first step (product in the first columns of S buffer 0, scaled and
// rounded to bf16 by the softmax threads).  The caches arrive by TMA into rings of stages
// guarded by mbarriers: one box per page and 64-column slab when a block table scatters the pages, one
// box per slab for the whole 128-token stage (4-D tensor map) when the pages are consecutive.
//
// TMEM columns: S0 [0,128) | S1 [128,256) | P [256,320) | O' [320, 320 + 192).  Because P does not
// overlay S, an S buffer is free as soon as the softmax threads have pulled it into registers, so
// Q K^T runs two steps ahead of the softmax; P has one buffer and is rewritten once the previous P V'
// has retired (that MMA was issued a whole step earlier).
//
// Warp roles: warp 0 = TMA producer of the key ring, the last warp = TMA producer of the value ring
// (keys are released right after S is computed, values only after O' is updated, so the two rings run
// at different distances ahead), warp 1 = TMEM owner + Q K^T issuer, warp 2 = P V' issuer (an MMA costs
// its issuing thread about a hundred cycles, so the two streams are issued by different threads), the
// 8 warps in between = softmax / correction / epilogue.  The row maximum of a step is taken one step
// ahead (in the middle of the previous step's exponentials) and the reference maximum is only raised
// when it grows by more than 8 (log2 domain), so O' is rescaled a handful of times per row instead of
// at every step; P stays below 2^8.  Every mbarrier wait is bounded and falls through with
// PRECC_STATUS_TIMEOUT.
//
// Two more instantiations of the same kernel.  VH: the value ring holds units of 64 tokens instead of whole
// steps (where one value stage fits beside two key stages but two do not), a unit being freed as soon as its
// four k-steps of P V' retire.  WL: the work-list launch - a 1-D grid in which the first (row tiles x kv heads)
// blocks stop `helper_p` steps into their tile and the remaining blocks share the tails of all tiles, several
// pieces each with the block drained in between; the pieces of a tile meet through fp32 records in a
// caller-provided workspace, and the block that arrives last at the tile's ticket merges them in piece order.
#pragma once
#include <type_traits>

#include "tc_common.cuh"

namespace precc {

struct PrefillTcParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int32_t* block_table;
  const __nv_bfloat16* B_k;    // already offset to the agent: [r_k][n_kv*hd]
  const __nv_bfloat16* B_v;
  uint32_t* status;
  int64_t n_blocks;
  int S, T, first_block;
  int n_q, n_kv, group;
  int tok_per_tile;            // 128 / group
  int k_stages, v_stages;      // depth of the key ring and of the value ring
  int v_half;                  // 1: the value ring holds v_stages units of 64 tokens (half a step) instead of whole steps - where
                               //    shared memory has room for one and a half value stages but not for two
  int contig;                  // 1: no block table; the tensor maps fetch a whole 128-token stage per box
  int k_logical;               // 1: the key map covers a scratch copy of this sequence's keys in logical block order (whole-stage boxes
                               //    from block 0), whatever the layout of the value side
  int longest_first;           // 1: block x = 0 takes the LAST row tile (longest causal reach), so the tail of the grid is short blocks
  float scale_log2, s_k, s_v;
  unsigned long long* trace;   // PRECC_PF_TRACE builds only: [steps][16] clock stamps of block (0, 0)
  // Work-list launch (helper_p > 0; 1-D grid of tiles + n_helpers blocks, no cluster): block b < tiles takes steps
  // [0, helper_p) of tile b, the n_helpers blocks behind them share the tails of all tiles; the pieces of a tile meet
  // through records in `ws_rec`, and the block that arrives last at the tile's ticket merges them.
  int helper_p, n_helpers, row_tiles;
  float* ws_rec;               // [2 * tiles + n_helpers][PrefillTcCfg::REC_FLOATS]
  unsigned int* ws_ticket;     // [tiles], zero before the launch and again after it
};

// Timeline stamps for tuning (compiled in with -DPRECC_PF_TRACE; slot meanings at the call sites).
#ifdef PRECC_PF_TRACE
#define PTC_STAMP(p, j, slot)                                                                    \
  do {                                                                                           \
    if ((p).trace && blockIdx.x == 0 && blockIdx.y == 0 && (j) < 64) (p).trace[(j) * 16 + (slot)] = clock64(); \
  } while (0)
// work-list launch: wall-clock stamps of every block's pieces (thread 0 of the softmax warps), behind the step stamps
#define PTC_WL_STAMP(p, seg, slot)                                                               \
  do {                                                                                           \
    if ((p).trace && (p).helper_p > 0 && threadIdx.x == PTC_FIRST_SM_WARP * 32 && (seg) < 16) {   \
      unsigned long long t__;                                                                    \
      asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t__));                                 \
      (p).trace[1024 + blockIdx.x * 128 + (seg) * 8 + (slot)] = t__;                             \
    }                                                                                            \
  } while (0)
#else
#define PTC_STAMP(p, j, slot) do { } while (0)
#define PTC_WL_STAMP(p, seg, slot) do { } while (0)
#endif

constexpr int PTC_PARTS_MAX = 4;
constexpr int PTC_PARTS = 2;                         // softmax threads per query row
constexpr int PTC_SOFTMAX_WARPS = 4 * PTC_PARTS;
constexpr int PTC_FIRST_SM_WARP = 3;                 // warps 0..2: key producer, QK^T issuer, PV issuer
constexpr int PTC_THREADS = (PTC_FIRST_SM_WARP + PTC_SOFTMAX_WARPS + 1) * 32;
constexpr int PTC_SMEM_LIMIT = 232448;   // dynamic shared memory a block can opt into on this architecture
constexpr int PTC_FIXED_BARS = 10; // barriers besides the two per ring stage
constexpr int PTC_TOK = 128;      // tokens per step
constexpr float PTC_RAISE = 8.f;  // the running maximum is raised only when it grows by more than this
constexpr int PTC_MAX_SRC = 8;    // work-list launch: pieces of one tile (its own block + helper pieces) at most
constexpr int PTC_MAX_SEG = 16;   // work-list launch: tile pieces one helper block takes at most
constexpr int PTC_MAX_XT = 160;   // work-list launch: row tiles at most
constexpr int PTC_TAB_BYTES = (2 * PTC_MAX_XT + 8 + 4 * PTC_MAX_SEG) * 4;   // tail lengths | their prefix sums | scalars | piece list

template <int HD, int RK, int RV>
struct PrefillTcCfg {
  static constexpr int SLABS = HD / 64;                      // 64-column slabs of a base row
  static constexpr int SLAB_BYTES = PTC_TOK * 128;            // 128 rows x 128 bytes
  static constexpr int Q_BYTES = SLABS * SLAB_BYTES;
  static constexpr int RKP = RK == 8 ? 16 : RK;               // rank 8 rides as a zero-padded k step of 16
  static constexpr int QX_BYTES = RK > 0 ? PTC_TOK * RKP * 2 : 0;
  static constexpr int KV_BYTES = SLABS * SLAB_BYTES;
  static constexpr int LK_BYTES = PTC_TOK * RKP * 2;
  static constexpr int LV_BYTES = PTC_TOK * RV * 2;
  static constexpr int KSTAGE = KV_BYTES + LK_BYTES;          // {K_base slabs | L_K} of 128 tokens
  static constexpr int VSLABS = SLABS + (RV > 0 ? 1 : 0);     // L_V rides as one more 64-column slab (zero padded)
  static constexpr int OW = VSLABS * 64;                      // columns of O' in TMEM: [O | U | padding]
  static constexpr int VSTAGE = VSLABS * SLAB_BYTES;          // {V_base slabs | L_V slab}
  static constexpr int K_PAGE_TX = PAGE * (HD + RKP) * 2;      // bytes one page contributes to a key stage
  static constexpr int V_PAGE_TX = PAGE * VSLABS * 128;
  static constexpr int SPLIT_XS = (HD + RV + 15) / 16 * 16 + 4;                // row stride (floats) of a partial in shared memory
  // split-context merge area (laid over the Q tile, the folded-query tile and the rings): partial | m | l | merged rows | weights | 1/l | B_v slice
  static constexpr int SPLIT_BYTES = (128 * SPLIT_XS + 256 + 64 * SPLIT_XS + 16 * 64 + 64) * 4 + RV * HD * 2;
  static constexpr int REC_FLOATS = 128 * SPLIT_XS + 256;     // a tile's partial in global memory: O' rows | m[128] | l[128]
  // work-list merge area (same place): merged rows | weights of up to PTC_MAX_SRC pieces | 1/l | B_v slice
  static constexpr int WS_MERGE_BYTES = (128 * SPLIT_XS + PTC_MAX_SRC * 128 + 128) * 4 + RV * HD * 2;
  static constexpr bool L_IN_MMA = RV > 0 && RV < 64;         // a spare column of the L_V slab carries the denominator
  static constexpr int TMEM_P = 2 * PTC_TOK;                  // packed bf16 P (64 columns) after the two S buffers
  static constexpr int TMEM_O = TMEM_P + PTC_TOK / 2;         // O' (at most 192 columns): 320 + 192 = 512
  __host__ __device__ static constexpr int smem_bytes(int ks, int vs, bool v_half = false) { return Q_BYTES + QX_BYTES + ks * KSTAGE + vs * (v_half ? VSTAGE / 2 : VSTAGE) + 320 + 2 * PTC_PARTS_MAX * 512 + PTC_TAB_BYTES + 1024; }
  // one whole value stage fits beside two key stages, two do not, three half-step units do (head_dim 128 with rank 64)
  static constexpr bool V_HALF_CAPABLE = smem_bytes(2, 2) > PTC_SMEM_LIMIT && smem_bytes(2, 1) <= PTC_SMEM_LIMIT && smem_bytes(2, 3, true) <= PTC_SMEM_LIMIT;
  static constexpr bool supported = (HD == 64 || HD == 128) && (RK == 0 || RK == 8 || RK == 16 || RK == 32 || RK == 64) &&
                                    (RV == 0 || RV == 8 || RV == 16 || RV == 32 || RV == 64);
};

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}

// layout_type field of a shared-memory matrix descriptor for rows of `row_bytes`
__device__ __forceinline__ constexpr uint64_t umma_layout_for(int row_bytes) {
  return row_bytes >= 128 ? 2ull : (row_bytes == 64 ? 4ull : 6ull);
}
// K-major operand: rows of `row_bytes` (one swizzle span), 8-row groups `8*row_bytes` apart.
__device__ __forceinline__ uint64_t umma_desc_kmajor(uint32_t saddr, int row_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFF) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>((8 * row_bytes) >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= umma_layout_for(row_bytes) << 61;
  return d;
}
// MN-major operand (rows = k index, `row_bytes` of contiguous MN elements per row): 8-row groups
// `8*row_bytes` apart (stride offset), successive MN blocks `mn_block_stride` bytes apart (leading offset).
__device__ __forceinline__ uint64_t umma_desc_mnmajor(uint32_t saddr, int row_bytes, int mn_block_stride) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFF) >> 4);
  d |= static_cast<uint64_t>((mn_block_stride >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>((8 * row_bytes) >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= umma_layout_for(row_bytes) << 61;
  return d;
}
// D fp32, A/B bf16, M = 128, N = n; b_mn = 1 when B is MN-major.
__device__ __forceinline__ uint32_t umma_idesc(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(b_mn) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}

// WL: the work-list form (helper blocks; a block takes a list of tile pieces).  It is a separate instantiation so that
// the classic launch carries none of its state through the step loop (the kernel sits at its register limit).
// VH: the value ring holds units of 64 tokens (half a step) - instantiated only where shared memory has room for
// one whole value stage but not for two.
template <int HD, int RK, int RV, bool WL = false, bool VH = false>
__global__ void __launch_bounds__(PTC_THREADS, 1)
lr_attend_prefill_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                            const __grid_constant__ CUtensorMap map_lk, const __grid_constant__ CUtensorMap map_lv,
                            const PrefillTcParams p) {
  using C = PrefillTcCfg<HD, RK, RV>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const uint32_t q_u32 = smem_u32(smem);
  const uint32_t qx_u32 = q_u32 + C::Q_BYTES;
  const uint32_t kring_u32 = qx_u32 + C::QX_BYTES;
  const int KS = p.k_stages, VS = p.v_stages;
  unsigned char* kring = smem + C::Q_BYTES + C::QX_BYTES;
  unsigned char* vring = kring + (size_t)KS * C::KSTAGE;
  const uint32_t vring_u32 = kring_u32 + KS * C::KSTAGE;
  constexpr bool v_half = VH;
  const int vunit = v_half ? C::VSTAGE / 2 : C::VSTAGE;   // bytes of one slot of the value ring
  uint64_t* bars = reinterpret_cast<uint64_t*>(vring + (size_t)VS * vunit);
  const uint32_t bar0 = smem_u32(bars);
  // barrier map: k_full[KS] | k_empty[KS] | v_full[VS] | v_empty[VS] | s_full[2] | p_full[2] | pv_done | q_ready | s_free[2] | fold_go | fold_done
  const uint32_t k_full = bar0, k_empty = k_full + 8 * KS, v_full = k_empty + 8 * KS, v_empty = v_full + 8 * VS,
                 s_full = v_empty + 8 * VS, p_full = s_full + 16, pv_done = p_full + 16, q_ready = pv_done + 8,
                 s_free = q_ready + 8, fold_go = s_free + 16, fold_done = fold_go + 8;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * KS + 2 * VS + PTC_FIXED_BARS);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.group;
  constexpr bool worklist = WL;
  // What this block works on.  Classic launch: one (row tile, kv head) per block, fixed for the whole kernel.  Work-list
  // launch: a short list of tile pieces, taken one after the other with the block drained in between.
  int g = blockIdx.y;
  int tok0 = (p.longest_first ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x) * p.tok_per_tile;
  int n_tok = min(p.tok_per_tile, p.S - tok0);             // new tokens handled by this block
  int t_end = p.T + tok0 + n_tok;                          // context + causal reach of the last row
  int full_vis = p.T + tok0 + 1;                           // tokens visible to every row of the block
  // Short turns over long contexts: the 128-token steps of a (row tile, kv head) are split over the NS
  // blocks of a cluster (grid/cluster z; any size from 2 to 8), each producing a partial (m, l, O') that the cluster merges
  // over distributed shared memory.  `jb` is this block's first step, `n_tiles` its number of steps
  // (possibly zero); loop indices below are local, token positions use jb + j.
  uint32_t split, NS;
  asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(split));
  asm volatile("mov.u32 %0, %%cluster_nctaid.z;\n" : "=r"(NS));
  int jb = 0, n_tiles = 0;
  if constexpr (!worklist) {
    const int n_total = (t_end + PTC_TOK - 1) / PTC_TOK;
    const int chunk_steps = (n_total + (int)NS - 1) / (int)NS;
    jb = min(n_total, (int)split * chunk_steps);
    n_tiles = min(n_total, jb + chunk_steps) - jb;
  }
  // work-list tables behind the maxima exchange area: tail[x] | pre[x] | scalars | pieces {tile, first step, steps, -}
  int* tab_tail = reinterpret_cast<int*>(bars + 2 * KS + 2 * VS + PTC_FIXED_BARS + 2) + 2 * PTC_PARTS_MAX * 128;
  int* tab_pre = tab_tail + PTC_MAX_XT;
  int* tab_sc = tab_pre + PTC_MAX_XT;                      // [0] pieces of this block, [1] sum of the tails of one kv head, [2] tail steps per helper
  int* tab_seg = tab_sc + 8;
  auto steps_of = [&](int x) { return (p.T + min(p.S, (x + 1) * p.tok_per_tile) + PTC_TOK - 1) / PTC_TOK; };

  auto init_bars = [&]() {
    for (int s = 0; s < KS; ++s) { mbar_init(k_full + 8 * s, 1); mbar_init(k_empty + 8 * s, 1); }
    for (int s = 0; s < VS; ++s) { mbar_init(v_full + 8 * s, 1); mbar_init(v_empty + 8 * s, 1); }
    mbar_init(s_full, 1); mbar_init(s_full + 8, 1);
    mbar_init(p_full, PTC_SOFTMAX_WARPS); mbar_init(p_full + 8, PTC_SOFTMAX_WARPS);
    mbar_init(pv_done, 1);
    mbar_init(s_free, PTC_SOFTMAX_WARPS); mbar_init(s_free + 8, PTC_SOFTMAX_WARPS);
    mbar_init(q_ready, PTC_SOFTMAX_WARPS);
    mbar_init(fold_go, PTC_SOFTMAX_WARPS); mbar_init(fold_done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    fence_async_smem();
  };
  if (threadIdx.x == 0) init_bars();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_holder)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if constexpr (worklist) {
    for (int x = threadIdx.x; x < p.row_tiles; x += blockDim.x) tab_tail[x] = max(0, steps_of(x) - p.helper_p);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const int n_base_tiles = p.row_tiles * p.n_kv;           // work-list launch: blocks below this index own a tile
  if constexpr (worklist) {
    if (threadIdx.x == 0) {
      const int X = p.row_tiles;
      int acc = 0;
      for (int x = 0; x < X; ++x) { tab_pre[x] = acc; acc += tab_tail[x]; }
      const int tail_sum = acc, total = acc * p.n_kv;
      const int per = max(1, (total + p.n_helpers - 1) / max(1, p.n_helpers));
      int n = 0;
      const int b = blockIdx.x;
      if (b < n_base_tiles) {
        const int x = b % X;
        tab_seg[0] = b; tab_seg[1] = 0; tab_seg[2] = steps_of(x) - tab_tail[x];
        n = 1;
      } else {
        const int h = b - n_base_tiles;
        int pos = min(total, h * per);
        const int hi = min(total, pos + per);
        if (pos < hi) {
          int gg = pos / tail_sum, off = pos - gg * tail_sum, x = 0;
          while (tab_pre[x] + tab_tail[x] <= off) ++x;
          while (pos < hi && n < PTC_MAX_SEG) {
            const int take = min(hi - pos, tab_pre[x] + tab_tail[x] - off);
            tab_seg[4 * n] = gg * X + x;
            tab_seg[4 * n + 1] = steps_of(x) - tab_tail[x] + (off - tab_pre[x]);
            tab_seg[4 * n + 2] = take;
            ++n; pos += take; off += take;
            while (x < X && tab_pre[x] + tab_tail[x] <= off) ++x;
            if (x == X) { ++gg; off = 0; x = 0; while (x < X - 1 && tab_tail[x] == 0) ++x; off = tab_pre[x]; }
          }
        }
      }
      tab_sc[0] = n; tab_sc[1] = tail_sum; tab_sc[2] = per;
    }
    __syncthreads();
  }
  const int nseg = worklist ? tab_sc[0] : 1;
  for (int seg = 0; seg < nseg; ++seg) {
  // work-list launch: the tile of this piece, where its record goes and which records make up the tile
  bool to_ws = false;
  int tile_u = 0, rec_id = 0, n_src = 1, src_first = 0;
  if constexpr (worklist) {
    tile_u = tab_seg[4 * seg]; jb = tab_seg[4 * seg + 1]; n_tiles = tab_seg[4 * seg + 2];
    const int x = tile_u % p.row_tiles;
    g = tile_u / p.row_tiles;
    tok0 = x * p.tok_per_tile;
    n_tok = min(p.tok_per_tile, p.S - tok0);
    t_end = p.T + tok0 + n_tok;
    full_vis = p.T + tok0 + 1;
    if (tab_tail[x] > 0) {
      const int a_u = g * tab_sc[1] + tab_pre[x], per = tab_sc[2];
      const int hf = a_u / per, hl = (a_u + tab_tail[x] - 1) / per;
      to_ws = true;
      n_src = 2 + hl - hf;
      src_first = n_base_tiles + tile_u + hf;              // record of the first helper piece; the tile's own block writes record tile_u
      rec_id = (int)blockIdx.x < n_base_tiles ? tile_u : n_base_tiles + tile_u + ((int)blockIdx.x - n_base_tiles);
    }
    if (seg > 0) {
      // the block is drained (every load consumed, every MMA retired, all threads past the barrier that ended the
      // previous piece): fresh barriers for the next piece
      if (threadIdx.x == 0) {
        for (int i = 0; i < 2 * KS + 2 * VS + PTC_FIXED_BARS; ++i) asm volatile("mbarrier.inval.shared::cta.b64 [%0];\n" ::"r"(bar0 + 8 * i) : "memory");
        init_bars();
      }
      __syncthreads();
    }
  }

  if (warp == 0 || warp == PTC_FIRST_SM_WARP + PTC_SOFTMAX_WARPS) {
    // ------------------------------------------------------------------ TMA producers (keys / values)
    const bool is_k = warp == 0;
    const int NS = is_k ? KS : VS;
    const uint32_t fullb = is_k ? k_full : v_full, emptyb = is_k ? k_empty : v_empty;
    if (v_half && !is_k) {
      // value ring in units of 64 tokens: two units per step, each freed as soon as its four k-steps of P V' retire
      constexpr int UT = PTC_TOK / 2, UPG = UT / PAGE, HSLAB = C::SLAB_BYTES / 2;
      for (int u = 0; u < 2 * n_tiles; ++u) {
        const int s = u % VS;
        if (u >= VS) mbar_wait(v_empty + 8 * s, ((u / VS) - 1) & 1, p.status);
        const int t0 = (2 * jb + u) * UT;
        const uint32_t st = vring_u32 + (uint32_t)s * (C::VSTAGE / 2);
        const uint32_t full = v_full + 8 * s;
        if (p.contig) {
          if (lane == 0) {
            mbar_expect_tx(full, UPG * C::V_PAGE_TX);
            const int blk0 = p.first_block + (2 * jb + u) * UPG;
#pragma unroll
            for (int sl = 0; sl < C::SLABS; ++sl) tma_load_4d(st + sl * HSLAB, &map_v, sl * 64, 0, g, blk0, full);
            if constexpr (RV > 0) tma_load_2d(st + C::SLABS * HSLAB, &map_lv, 0, blk0 * PAGE, full);
          }
          __syncwarp();
          continue;
        }
        const int live = max(0, min(UPG, (t_end - t0 + PAGE - 1) / PAGE));
        if (lane == 0) mbar_expect_tx(full, live * C::V_PAGE_TX);       // no live page: the phase completes at once
        __syncwarp();
        if (lane < live) {
          const int lt = (2 * jb + u) * UPG + lane;
          int ph = p.block_table ? __ldg(p.block_table + lt) : p.first_block + lt;
          if (ph < 0 || ph >= p.n_blocks) { atomicOr(p.status, StatusBits::BAD_INDEX); ph = 0; }
          const int row_kv = (ph * p.n_kv + g) * PAGE;
#pragma unroll
          for (int sl = 0; sl < C::SLABS; ++sl) tma_load_2d(st + sl * HSLAB + lane * PAGE * 128, &map_v, sl * 64, row_kv, full);
          if constexpr (RV > 0) tma_load_2d(st + C::SLABS * HSLAB + lane * PAGE * 128, &map_lv, 0, ph * PAGE, full);
        }
        __syncwarp();
      }
    } else
    for (int j = 0; j < n_tiles; ++j) {
      const int s = j % NS;
      if (j >= NS) mbar_wait(emptyb + 8 * s, ((j / NS) - 1) & 1, p.status);
      // the last key stage doubles as the staging area of B_k until the query fold is done
      if (RK > 0 && is_k && j == KS - 1) mbar_wait(q_ready, 0, p.status);
      if (lane == 0) PTC_STAMP(p, j, is_k ? 8 : 9);               // stage of step j free: loads go out now
      const int t0 = (jb + j) * PTC_TOK;
      const int live = min(PTC_TOK / PAGE, (t_end - t0 + PAGE - 1) / PAGE);
      const uint32_t st = is_k ? kring_u32 + (uint32_t)s * C::KSTAGE : vring_u32 + (uint32_t)s * C::VSTAGE;
      const uint32_t full = fullb + 8 * s;
      if (p.contig || (is_k && p.k_logical)) {
        // consecutive physical blocks: one box per 64-column slab covers all eight pages of the stage
        // (4-D map [block][kv head][16][hd]); blocks past the cache end arrive as zeros
        if (lane == 0) {
          mbar_expect_tx(full, (PTC_TOK / PAGE) * (is_k ? C::K_PAGE_TX : C::V_PAGE_TX));
          const int blk0 = ((is_k && p.k_logical) ? 0 : p.first_block) + (jb + j) * (PTC_TOK / PAGE);
          if (is_k) {
#pragma unroll
            for (int sl = 0; sl < C::SLABS; ++sl) tma_load_4d(st + sl * C::SLAB_BYTES, &map_k, sl * 64, 0, g, blk0, full);
            if constexpr (RK > 0) tma_load_2d(st + C::KV_BYTES, &map_lk, 0, blk0 * PAGE, full);
          } else {
#pragma unroll
            for (int sl = 0; sl < C::SLABS; ++sl) tma_load_4d(st + sl * C::SLAB_BYTES, &map_v, sl * 64, 0, g, blk0, full);
            if constexpr (RV > 0) tma_load_2d(st + C::SLABS * C::SLAB_BYTES, &map_lv, 0, blk0 * PAGE, full);
          }
        }
        __syncwarp();
        continue;
      }
      if (lane == 0) mbar_expect_tx(full, live * (is_k ? C::K_PAGE_TX : C::V_PAGE_TX));
      __syncwarp();
      if (lane < live) {
        const int lt = (jb + j) * (PTC_TOK / PAGE) + lane;
        int ph = p.block_table ? __ldg(p.block_table + lt) : p.first_block + lt;
        if (ph < 0 || ph >= p.n_blocks) { atomicOr(p.status, StatusBits::BAD_INDEX); ph = 0; }
        const int row_kv = (ph * p.n_kv + g) * PAGE;
        if (is_k) {
#pragma unroll
          for (int sl = 0; sl < C::SLABS; ++sl) tma_load_2d(st + sl * C::SLAB_BYTES + lane * PAGE * 128, &map_k, sl * 64, row_kv, full);
          if constexpr (RK > 0) tma_load_2d(st + C::KV_BYTES + lane * PAGE * C::RKP * 2, &map_lk, 0, ph * PAGE, full);
        } else {
#pragma unroll
          for (int sl = 0; sl < C::SLABS; ++sl) tma_load_2d(st + sl * C::SLAB_BYTES + lane * PAGE * 128, &map_v, sl * 64, row_kv, full);
          if constexpr (RV > 0) tma_load_2d(st + C::SLABS * C::SLAB_BYTES + lane * PAGE * 128, &map_lv, 0, ph * PAGE, full);
        }
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ S = Q' K'^T issuer
    // One thread issues these MMAs and another (warp 2) the P V' ones: an MMA costs its issuing thread
    // on the order of a hundred cycles, so two issue streams are needed to keep the tensor pipe fed.
    // All descriptors are prepared once (the address field holds addr >> 4, so moving to another
    // stage, slab or k-step is one 64-bit add of a small constant).
    const uint32_t id_s = umma_idesc(PTC_TOK, 0);
    const uint64_t qd0 = umma_desc_kmajor(q_u32, 128);
    const uint64_t qxd0 = RK > 0 ? umma_desc_kmajor(qx_u32, C::RKP * 2) : 0;
    const uint64_t kd0 = umma_desc_kmajor(kring_u32, 128);
    const uint64_t lkd0 = RK > 0 ? umma_desc_kmajor(kring_u32 + C::KV_BYTES, C::RKP * 2) : 0;
    if constexpr (RK > 0) {
      // the key-side fold Q B_k^T (128 x RKP x HD): Q tile and B_k slice are staged, the product lands in the first
      // columns of S buffer 0, from where the softmax threads scale it into the folded-query tile
      mbar_wait(fold_go, 0, p.status);
      tc_fence_after();
      if (lane == 0) {
        const uint32_t id_f = umma_idesc(C::RKP, 0);
        const uint64_t bd0 = umma_desc_kmajor(kring_u32 + (uint32_t)(KS - 1) * C::KSTAGE, 128);
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint64_t qo = (uint64_t)(((ks / 4) * C::SLAB_BYTES + (ks % 4) * 32) >> 4);
          const uint64_t bo = (uint64_t)(((ks / 4) * (C::RKP * 128) + (ks % 4) * 32) >> 4);
          umma_bf16(tmem_base, qd0 + qo, bd0 + bo, id_f, ks ? 1u : 0u);
        }
        umma_commit(fold_done);
      }
      __syncwarp();
    }
    mbar_wait(q_ready, 0, p.status);
    for (int j = 0; j < n_tiles; ++j) {
      const int s = j % KS;
      // S buffer j&1 is free once the softmax threads have pulled the scores of step j-2 into registers
      // (P has its own columns), so Q K^T runs up to two steps ahead of the softmax
      if (j >= 2) mbar_wait(s_free + 8 * (j & 1), ((j >> 1) - 1) & 1, p.status);
      mbar_wait(k_full + 8 * s, (j / KS) & 1, p.status);
      tc_fence_after();
      if (lane == 0) {
        PTC_STAMP(p, j, 10);                     // keys of step j have landed (seen by the issuer)
        const uint64_t so = (uint64_t)((s * C::KSTAGE) >> 4);
        const uint32_t d = tmem_base + (j & 1) * PTC_TOK;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint64_t off = (uint64_t)(((ks / 4) * C::SLAB_BYTES + (ks % 4) * 32) >> 4);
          umma_bf16(d, qd0 + off, kd0 + so + off, id_s, ks ? 1u : 0u);
        }
        if constexpr (RK > 0) {
#pragma unroll
          for (int ks = 0; ks < C::RKP / 16; ++ks) umma_bf16(d, qxd0 + (uint64_t)(ks * 2), lkd0 + so + (uint64_t)(ks * 2), id_s, 1u);
        }
        umma_commit(k_empty + 8 * s);            // the key stage is free as soon as S is computed
        umma_commit(s_full + 8 * (j & 1));
        PTC_STAMP(p, j, 2);                      // QK^T of step j issued
      }
      __syncwarp();
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ O' += P V' issuer
    const uint32_t id_o = umma_idesc(C::OW, 1);
    const uint64_t vd0 = umma_desc_mnmajor(vring_u32, 128, C::SLAB_BYTES);
    if constexpr (v_half) {
      constexpr int UT = PTC_TOK / 2, HSLAB = C::SLAB_BYTES / 2;
      const uint64_t vdh = umma_desc_mnmajor(vring_u32, 128, HSLAB);
      for (int j = 0; j < n_tiles; ++j) {
        const int n_live = min(PTC_TOK, t_end - (jb + j) * PTC_TOK);     // tokens of this step that exist
        for (int half = 0; half < 2; ++half) {
          const int u = 2 * j + half, s = u % VS;
          const int live_u = max(0, min(UT, n_live - half * UT));        // tokens of this unit that exist
          mbar_wait(v_full + 8 * s, (u / VS) & 1, p.status);
          unsigned char* ub = vring + (size_t)s * (C::VSTAGE / 2);
          if constexpr (C::L_IN_MMA) {
            unsigned char* slab = ub + C::SLABS * HSLAB;
            constexpr int CH = (RV * 2) / 16;
            for (int r = lane; r < UT; r += 32)
              *reinterpret_cast<__nv_bfloat16*>(slab + r * 128 + ((CH ^ (r & 7)) * 16)) = __float2bfloat16(r < live_u ? 1.f : 0.f);
            fence_async_smem();
            __syncwarp();
          }
          if (live_u < UT && (p.contig || (live_u % PAGE) != 0)) {
            // rows past the end may hold anything: clear them before the MMA reads the unit
            const int r1 = p.contig ? UT : (live_u + PAGE - 1) / PAGE * PAGE;
            for (int r = live_u; r < r1; ++r)
              for (int sl = 0; sl < C::VSLABS; ++sl)
                for (int c = lane; c < 8; c += 32) *reinterpret_cast<uint4*>(ub + sl * HSLAB + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
            fence_async_smem();
            __syncwarp();
          }
          if (half == 0) mbar_wait(p_full + 8 * (j & 1), (j >> 1) & 1, p.status);
          tc_fence_after();
          if (lane == 0) {
            const uint32_t a = tmem_base + C::TMEM_P + half * (UT / 2);  // packed bf16 P, 2 per column
            const uint64_t so = (uint64_t)((s * (C::VSTAGE / 2)) >> 4);
            const uint32_t od = tmem_base + C::TMEM_O;
            const int n_ks = (live_u + 15) / 16;
            for (int ks = 0; ks < n_ks; ++ks) umma_bf16_ts(od, a + ks * 8, vdh + so + (uint64_t)(ks * 128), id_o, (j | half | ks) ? 1u : 0u);
            umma_commit(v_empty + 8 * s);
            if (half == 1) umma_commit(pv_done);
          }
          __syncwarp();
        }
      }
    } else
    for (int j = 0; j < n_tiles; ++j) {
      const int s = j % VS;
      const int n_live = min(PTC_TOK, t_end - (jb + j) * PTC_TOK);       // tokens of this step that exist
      mbar_wait(v_full + 8 * s, (j / VS) & 1, p.status);
      if (lane == 0) PTC_STAMP(p, j, 11);                          // values of step j have landed
      if constexpr (C::L_IN_MMA) {
        // column RV of the zero-padded L_V slab is set to one for the live tokens: the P V' MMA then
        // accumulates the softmax denominator sum_t p_t in column HD + RV of O' (same bf16 p as the numerator)
        unsigned char* slab = vring + (size_t)s * C::VSTAGE + C::SLABS * C::SLAB_BYTES;
        constexpr int CH = (RV * 2) / 16;                          // 16-byte chunk holding column RV
        for (int r = lane; r < PTC_TOK; r += 32)
          *reinterpret_cast<__nv_bfloat16*>(slab + r * 128 + ((CH ^ (r & 7)) * 16)) = __float2bfloat16(r < n_live ? 1.f : 0.f);
        fence_async_smem();
        __syncwarp();
      }
      if (n_live < PTC_TOK && (p.contig || (n_live % PAGE) != 0)) {
        // value rows past the end may hold anything (the rest of a partly written page; with whole-stage
        // boxes also the pages behind it), and 0 * NaN would poison the accumulators: clear them
        // before the MMA reads the stage
        const int r0 = n_live, r1 = p.contig ? PTC_TOK : (n_live + PAGE - 1) / PAGE * PAGE;
        unsigned char* base = vring + (size_t)s * C::VSTAGE;
        for (int r = r0; r < r1; ++r)
          for (int sl = 0; sl < C::VSLABS; ++sl)
            for (int c = lane; c < 8; c += 32) *reinterpret_cast<uint4*>(base + sl * C::SLAB_BYTES + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
        fence_async_smem();
        __syncwarp();
      }
      mbar_wait(p_full + 8 * (j & 1), (j >> 1) & 1, p.status);
      tc_fence_after();
      if (lane == 0) {
        PTC_STAMP(p, j, 0);                                        // P of step j seen by the PV issuer
        const uint32_t a = tmem_base + C::TMEM_P;                  // packed bf16 P, 2 per column
        const uint64_t so = (uint64_t)((s * C::VSTAGE) >> 4);
        const uint32_t od = tmem_base + C::TMEM_O;
        if (n_live == PTC_TOK) {
#pragma unroll
          for (int ks = 0; ks < PTC_TOK / 16; ++ks) umma_bf16_ts(od, a + ks * 8, vd0 + so + (uint64_t)(ks * 128), id_o, (j | ks) ? 1u : 0u);
        } else {
          const int n_ks = (n_live + 15) / 16;
          for (int ks = 0; ks < n_ks; ++ks) umma_bf16_ts(od, a + ks * 8, vd0 + so + (uint64_t)(ks * 128), id_o, (j | ks) ? 1u : 0u);
        }
        umma_commit(v_empty + 8 * s);
        umma_commit(pv_done);
        PTC_STAMP(p, j, 1);                                        // P V' of step j issued
      }
      __syncwarp();
    }
  } else if (warp >= PTC_FIRST_SM_WARP && warp < PTC_FIRST_SM_WARP + PTC_SOFTMAX_WARPS) {
    // ------------------------------------------------------------------ softmax / correction / epilogue
    // PTC_PARTS threads per query row, each owning 128/PTC_PARTS tokens of a step (a warp may only touch
    // the TMEM lane quadrant warp % 4, so the threads of a row sit in warps whose ids agree modulo 4).
    // Several warps per scheduler let one warp's exponentials overlap another's TMEM traffic.
    constexpr int NP = PTC_PARTS;
    constexpr int COLS = PTC_TOK / NP;                            // score columns per thread (32)
    constexpr int NSM = PTC_SOFTMAX_WARPS * 32;                   // softmax threads
    PTC_WL_STAMP(p, seg, 0);                                       // piece starts
    const int quad = warp & 3;                                    // TMEM lane quadrant this warp may touch
    const int part = (warp - PTC_FIRST_SM_WARP) >> 2;             // which tokens / which output columns
    const int row = quad * 32 + lane;                             // query row of this thread
    const int tid = (warp - PTC_FIRST_SM_WARP) * 32 + lane;
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const int i_new = tok0 + row / G, hg = row % G;
    const bool row_ok = row < n_tok * G;
    const int lim = row_ok ? p.T + i_new : -1;                    // last visible token of this row
    float* xch = reinterpret_cast<float*>(bars + 2 * KS + 2 * VS + PTC_FIXED_BARS + 2);   // [2][NP][128] row maxima exchanged by a row's threads
    auto row_sync = [&]() { asm volatile("bar.sync %0, %1;\n" ::"r"(2 + quad), "r"(32 * NP) : "memory"); };
    // ---- B_k slice into the last key stage and the Q rows into their tile, both as K-major swizzled operands; the
    //      fold Q~ = s_k Q B_k^T is one small MMA chain (issued by warp 1), scaled and rounded here
    unsigned char* bk_s = kring + (size_t)(KS - 1) * C::KSTAGE;
    if constexpr (RK > 0) {
      for (int c = tid; c < C::RKP * (HD / 8); c += NSM) {
        const int j = c / (HD / 8), ch = c % (HD / 8);
        const uint4 v = j < RK ? __ldg(reinterpret_cast<const uint4*>(p.B_k + (size_t)j * p.n_kv * HD + (size_t)g * HD + ch * 8))
                               : make_uint4(0u, 0u, 0u, 0u);    // rank 8 rides as a zero-padded step of 16
        *reinterpret_cast<uint4*>(bk_s + (ch / 8) * (C::RKP * 128) + j * 128 + (((ch % 8) ^ (j & 7)) * 16)) = v;
      }
    }
    {
      const uint4* src = reinterpret_cast<const uint4*>(p.q + ((size_t)i_new * p.n_q + (size_t)g * G + hg) * HD);
#pragma unroll
      for (int c = 0; c < HD / 8; ++c) {
        if ((c % NP) == part) {
          const int sl = c / 8, ch = c % 8;
          *reinterpret_cast<uint4*>(smem + sl * C::SLAB_BYTES + row * 128 + ((ch ^ (row & 7)) * 16)) =
              row_ok ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
        }
      }
      if constexpr (RK > 0) {
        constexpr int CPR = C::RKP / 8;
        fence_async_smem();                                       // the staged operands -> visible to the MMA unit
        __syncwarp();
        if (lane == 0) mbar_arrive(fold_go);
        mbar_wait(fold_done, 0, p.status);
        tc_fence_after();
#pragma unroll 1
        for (int c = part; c < C::RKP / 16; c += NP) {             // 16 coordinates per pass
          uint32_t fv[16];
          tmem_ld16(lane_addr + c * 16, fv);
          tmem_wait_ld();
          uint32_t pk[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) pk[k] = pack_bf16(__uint_as_float(fv[2 * k]) * p.s_k, __uint_as_float(fv[2 * k + 1]) * p.s_k);
          *reinterpret_cast<uint4*>(smem + C::Q_BYTES + swz_off<CPR>(row, 2 * c)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          *reinterpret_cast<uint4*>(smem + C::Q_BYTES + swz_off<CPR>(row, 2 * c + 1)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        }
        tc_fence_before();                                        // the reads of S buffer 0 precede the first Q K^T
      }
    }
    fence_async_smem();                                           // generic-proxy writes -> visible to the MMA unit
    __syncwarp();
    if (lane == 0) mbar_arrive(q_ready);
    PTC_WL_STAMP(p, seg, 1);                                       // query tile loaded and folded

    constexpr int OCH = (HD + RV) / 16 + (C::L_IN_MMA ? 1 : 0);   // 16-column chunks of O' that carry data (numerator, U, denominator)
    float m_used = NEG_BIG, l_sum = 0.f;
    constexpr int NCH = COLS / 32;
    // This thread's maximum (log2 domain) over its COLS scores of step j, read straight from TMEM.  It is
    // taken one step ahead, in the middle of the previous step's exponentials, so that its latency chain
    // (TMEM read, compare chain, exchange between the row's threads) is off the critical path.
    auto local_max = [&](int j) -> float {
      const int b = j & 1;
      const int nvis = lim - ((jb + j) * PTC_TOK + part * COLS) + 1;   // visible tokens among this thread's
      const bool masked = (jb + j) * PTC_TOK + PTC_TOK > full_vis;
      float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        uint32_t x[32];
        tmem_ld32(lane_addr + b * PTC_TOK + part * COLS + c * 32, x);
        tmem_wait_ld();
        if (masked) {
#pragma unroll
          for (int k = 0; k < 32; ++k)
            if (c * 32 + k >= nvis) x[k] = 0xff800000u;          // -inf
        }
#pragma unroll
        for (int k = 0; k < 32; k += 2)                            // two elements per step: the three-input maximum
          tm[(k >> 1) & 3] = fmaxf(tm[(k >> 1) & 3], fmaxf(__uint_as_float(x[k]), __uint_as_float(x[k + 1])));
      }
      return fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])) * p.scale_log2;
    };
    // row maximum from the per-thread maxima of the row's NP threads
    auto exchange_max = [&](int j, float own) -> float {
      const int b = j & 1;
      xch[(b * NP + part) * 128 + row] = own;
      row_sync();
      float t = own;
#pragma unroll
      for (int q2 = 0; q2 < NP; ++q2) t = fmaxf(t, xch[(b * NP + q2) * 128 + row]);
      return t;
    };
    float tmax = NEG_BIG;                                         // row maximum of the step about to run
    // One step of the online softmax for this thread's COLS scores.  MASKED is a compile-time flag so
    // that the common step (far from the causal edge) carries no per-element compare/select.
    auto step = [&](int j, auto masked_tag) {
      constexpr bool MASKED = decltype(masked_tag)::value;
      const int b = j & 1;
      uint32_t sv[NCH][32];
#pragma unroll
      for (int c = 0; c < NCH; ++c) tmem_ld32(lane_addr + b * PTC_TOK + part * COLS + c * 32, sv[c]);
      tmem_wait_ld();
      if (tid == 0) PTC_STAMP(p, j, 7);                            // scores in registers
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_free + 8 * b);                  // the S buffer may be overwritten
      if constexpr (MASKED) {
        const int nvis = lim - ((jb + j) * PTC_TOK + part * COLS) + 1;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
          for (int k = 0; k < 32; ++k)
            if (c * 32 + k >= nvis) sv[c][k] = 0xff800000u;      // -inf: weight zero
      }
      // The two warps of a row share a scheduler and its special-function unit.  They take the next step's maximum at
      // different points of the step - one here, one between the halves of its exponentials - so that one warp's
      // exponentials run while the other reads tensor memory and compares, instead of both queueing for the unit at once.
      float next_own = NEG_BIG;
      const bool max_first = !VH && part == 1;                     // (with the half-step value ring the skew measured slower)
      if (max_first && j + 1 < n_tiles) {
        mbar_wait(s_full + 8 * ((j + 1) & 1), ((j + 1) >> 1) & 1, p.status);
        tc_fence_after();
        next_own = local_max(j + 1);
      }
      float m_new = m_used;
      if (tmax > m_used + PTC_RAISE) m_new = tmax;                 // all threads of the row decide alike
      const bool raise = m_new != m_used;
      if (__any_sync(0xffffffffu, raise)) {
        const float alpha = fast_exp2(m_used - m_new);             // 1 for rows that keep their maximum
        if (j > 0) {
          mbar_wait(pv_done, (j - 1) & 1, p.status);               // O' is complete through step j-1
          tc_fence_after();
#pragma unroll 1
          for (int c = part; c < OCH; c += NP) {
            uint32_t ov[16];
            tmem_ld16(lane_addr + C::TMEM_O + c * 16, ov);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 16; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * alpha);
            tmem_st16(lane_addr + C::TMEM_O + c * 16, ov);
          }
          tmem_wait_st();
        }
        l_sum *= alpha;
        m_used = m_new;
      }
      if (tid == 0) PTC_STAMP(p, j, 5);                            // reference maximum settled
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
      const float neg_m = -m_used;
      uint32_t pk[NCH][16];
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
#pragma unroll
        for (int k = 0; k < 32; k += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(sv[c][k]), p.scale_log2, neg_m));
          const float p1 = fast_exp2(fmaf(__uint_as_float(sv[c][k + 1]), p.scale_log2, neg_m));
          if constexpr (!C::L_IN_MMA) ls[(k >> 1) & 3] += p0 + p1;
          pk[c][k / 2] = pack_bf16(p0, p1);
        }
        if (c == 0 && !max_first && j + 1 < n_tiles) {
          if (tid == 0) PTC_STAMP(p, j, 12);                       // first half of the exponentials done
          // between the two halves of the exponentials: the next step's scores are normally there already
          mbar_wait(s_full + 8 * ((j + 1) & 1), ((j + 1) >> 1) & 1, p.status);
          tc_fence_after();
          next_own = local_max(j + 1);
          if (tid == 0) PTC_STAMP(p, j, 13);                       // next step's local maximum taken
        }
      }
      l_sum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      // P has one buffer: it may be overwritten once the previous step's P V' has read it (that MMA was
      // issued a whole softmax step ago, so this wait normally falls through)
      if (tid == 0) PTC_STAMP(p, j, 14);                           // all exponentials done
      if (j > 0) { mbar_wait(pv_done, (j - 1) & 1, p.status); tc_fence_after(); }
      if (tid == 0) PTC_STAMP(p, j, 15);                           // previous P V' has retired
#pragma unroll
      for (int c = 0; c < NCH; ++c) tmem_st16(lane_addr + C::TMEM_P + part * (COLS / 2) + c * 16, pk[c]);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full + 8 * b);
      if (tid == 0) PTC_STAMP(p, j, 6);                            // P published
      if (j + 1 < n_tiles) tmax = exchange_max(j + 1, next_own);
    };
    if (tid == 0) PTC_STAMP(p, 0, 3);
    if (n_tiles > 0) {
      mbar_wait(s_full, 0, p.status);
      tc_fence_after();
      tmax = exchange_max(0, local_max(0));
    }
    PTC_WL_STAMP(p, seg, 2);                                       // first scores seen
    for (int j = 0; j < n_tiles; ++j) {
      if (tid == 0) PTC_STAMP(p, j, 4);                            // step j starts (its scores were awaited a step earlier)
      if ((jb + j) * PTC_TOK + PTC_TOK > full_vis) step(j, std::true_type{});   // only the last few steps reach the causal edge
      else step(j, std::false_type{});
      if (tid == 0) PTC_STAMP(p, j + 1, 3);
    }
    // ---- epilogue: out = (O + s_v U B_v) / l ; the threads of a row share its output columns
    if (n_tiles > 0) { mbar_wait(pv_done, (n_tiles - 1) & 1, p.status); tc_fence_after(); }
    PTC_WL_STAMP(p, seg, 3);                                       // all steps done
    if (NS > 1) {
      // ---- split context: this block's partial (m, l, O') goes to shared memory for the cluster merge below
      constexpr int XS = C::SPLIT_XS;
      float* xo = reinterpret_cast<float*>(smem);          // the merge area starts at the Q tile: every MMA has completed
      float* xm = xo + 128 * XS;
      float* xl = xm + 128;
      float l_loc = 0.f;
      if constexpr (!C::L_IN_MMA) {
        xch[part * 128 + row] = l_sum;
        asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
#pragma unroll
        for (int q2 = 0; q2 < NP; ++q2) l_loc += xch[q2 * 128 + row];
      } else if (n_tiles > 0) {
        uint32_t lv16[16];
        tmem_ld16(lane_addr + C::TMEM_O + HD + (RV / 16) * 16, lv16);
        tmem_wait_ld();
        l_loc = __uint_as_float(lv16[RV % 16]);
      }
#pragma unroll 1
      for (int c = part; c < (HD + RV + 15) / 16; c += NP) {
        uint32_t ov[16];
        if (n_tiles > 0) {
          tmem_ld16(lane_addr + C::TMEM_O + c * 16, ov);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) ov[k] = 0u;
        }
#pragma unroll
        for (int k = 0; k < 16; k += 4)
          *reinterpret_cast<uint4*>(xo + row * XS + c * 16 + k) = make_uint4(ov[k], ov[k + 1], ov[k + 2], ov[k + 3]);
      }
      if (part == 0) { xm[row] = n_tiles > 0 ? m_used : NEG_BIG; xl[row] = n_tiles > 0 ? l_loc : 0.f; }
    } else if (WL && to_ws) {
      // ---- work-list launch: this piece's partial (m, l, O') goes to its record in global memory; the block that
      //      arrives last at the tile's ticket merges the tile's records in a fixed order and writes the output
      constexpr int XS = C::SPLIT_XS;
      float* rec = p.ws_rec + (size_t)rec_id * C::REC_FLOATS;
      float l_loc = 0.f;
      if constexpr (!C::L_IN_MMA) {
        xch[part * 128 + row] = l_sum;
        asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
#pragma unroll
        for (int q2 = 0; q2 < NP; ++q2) l_loc += xch[q2 * 128 + row];
      } else {
        uint32_t lv16[16];
        tmem_ld16(lane_addr + C::TMEM_O + HD + (RV / 16) * 16, lv16);
        tmem_wait_ld();
        l_loc = __uint_as_float(lv16[RV % 16]);
      }
#pragma unroll 1
      for (int c = part; c < (HD + RV + 15) / 16; c += NP) {
        uint32_t ov[16];
        tmem_ld16(lane_addr + C::TMEM_O + c * 16, ov);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 16; k += 4)
          __stcg(reinterpret_cast<uint4*>(rec + row * XS + c * 16 + k), make_uint4(ov[k], ov[k + 1], ov[k + 2], ov[k + 3]));
      }
      if (part == 0) { __stcg(rec + 128 * XS + row, m_used); __stcg(rec + 128 * XS + 128 + row, l_loc); }
      __threadfence();
      PTC_WL_STAMP(p, seg, 4);                                     // record written
      asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
      int* flag = reinterpret_cast<int*>(xch) + 2 * PTC_PARTS_MAX * 128 - 1;   // last word of the exchange area
      if (tid == 0) *flag = (int)atomicAdd(p.ws_ticket + tile_u, 1u);
      asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
      if (*flag == n_src - 1) {
        __threadfence();
        // merge area over the Q tile and the rings: every load of this piece has been consumed, every MMA has retired
        float* mo = reinterpret_cast<float*>(smem);         // merged rows [128][XS]
        float* wts = mo + 128 * XS;                         // [n_src][128] weights of the pieces
        float* linv = wts + PTC_MAX_SRC * 128;              // [128]
        unsigned char* bvs = reinterpret_cast<unsigned char*>(linv + 128);   // B_v[:, g] slice, [RV][HD] bf16
        auto src = [&](int k) -> const float* {
          return p.ws_rec + (size_t)(k == 0 ? tile_u : src_first + k - 1) * C::REC_FLOATS;
        };
        if constexpr (RV > 0) {
          for (int c = tid; c < RV * (HD / 8); c += NSM) {
            const int j = c / (HD / 8), ch = c % (HD / 8);
            *reinterpret_cast<uint4*>(bvs + (j * HD + ch * 8) * 2) =
                __ldg(reinterpret_cast<const uint4*>(p.B_v + (size_t)j * p.n_kv * HD + (size_t)g * HD + ch * 8));
          }
        }
        if (tid < 128) {
          float ms[PTC_MAX_SRC], M = NEG_BIG, L = 0.f;
#pragma unroll
          for (int k = 0; k < PTC_MAX_SRC; ++k) { ms[k] = k < n_src ? __ldcg(src(k) + 128 * XS + tid) : NEG_BIG; M = fmaxf(M, ms[k]); }
#pragma unroll
          for (int k = 0; k < PTC_MAX_SRC; ++k) {
            if (k < n_src) {
              const float wv = fast_exp2(ms[k] - M);
              wts[k * 128 + tid] = wv;
              L += wv * __ldcg(src(k) + 128 * XS + 128 + tid);       // piece order: deterministic
            }
          }
          linv[tid] = L > 0.f ? 1.f / L : 0.f;
        }
        asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
        constexpr int F4 = (HD + RV) / 4;                   // float4 columns of a merged row
        constexpr int UN = 8;                               // items per thread in flight: the records come from L2
        for (int it0 = tid; it0 < 128 * F4; it0 += NSM * UN) {
          float4 acc[UN];
#pragma unroll
          for (int u = 0; u < UN; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int k = 0; k < n_src; ++k) {
            const float* sk = src(k);
            float4 x[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) {
              const int it = it0 + u * NSM;
              x[u] = it < 128 * F4 ? __ldcg(reinterpret_cast<const float4*>(sk + (it / F4) * XS + (it % F4) * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < UN; ++u) {
              const int it = it0 + u * NSM;
              const float wv = it < 128 * F4 ? wts[k * 128 + it / F4] : 0.f;
              acc[u].x += wv * x[u].x; acc[u].y += wv * x[u].y; acc[u].z += wv * x[u].z; acc[u].w += wv * x[u].w;
            }
          }
#pragma unroll
          for (int u = 0; u < UN; ++u) {
            const int it = it0 + u * NSM;
            if (it < 128 * F4) *reinterpret_cast<float4*>(mo + (it / F4) * XS + (it % F4) * 4) = acc[u];
          }
        }
        asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
        // out = (O + s_v U B_v) / l, eight columns per item
        for (int it = tid; it < 128 * (HD / 8); it += NSM) {
          const int rl = it / (HD / 8), c8 = (it % (HD / 8)) * 8;
          if (rl >= n_tok * G) continue;
          float o[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) o[k] = mo[rl * XS + c8 + k];
          if constexpr (RV > 0) {
#pragma unroll 4
            for (int jv = 0; jv < RV; ++jv) {
              const float uj = mo[rl * XS + HD + jv] * p.s_v;
              const uint4 y = *reinterpret_cast<const uint4*>(bvs + (jv * HD + c8) * 2);
              const uint32_t ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                o[2 * k] += uj * bf16_bits_to_float(ys[k] & 0xffff);
                o[2 * k + 1] += uj * bf16_bits_to_float(ys[k] >> 16);
              }
            }
          }
          const float inv = linv[rl];
          const int i_out = tok0 + rl / G, h_out = rl % G;
          uint4 w;
          w.x = pack_bf16(o[0] * inv, o[1] * inv); w.y = pack_bf16(o[2] * inv, o[3] * inv);
          w.z = pack_bf16(o[4] * inv, o[5] * inv); w.w = pack_bf16(o[6] * inv, o[7] * inv);
          *reinterpret_cast<uint4*>(p.out + ((size_t)i_out * p.n_q + (size_t)g * G + h_out) * HD + c8) = w;
        }
        if (tid == 0) p.ws_ticket[tile_u] = 0u;             // the workspace is ready for the next call
        PTC_WL_STAMP(p, seg, 6);                                   // merged and stored
      }
      PTC_WL_STAMP(p, seg, 5);                                     // piece ends
    } else {
    unsigned char* bv_s = vring;                                  // value stage 0 is free now
    if constexpr (RV > 0) {
      for (int c = tid; c < RV * (HD / 8); c += NSM) {
        const int j = c / (HD / 8), ch = c % (HD / 8);
        *reinterpret_cast<uint4*>(bv_s + (j * HD + ch * 8) * 2) =
            __ldg(reinterpret_cast<const uint4*>(p.B_v + (size_t)j * p.n_kv * HD + (size_t)g * HD + ch * 8));
      }
    }
    xch[part * 128 + row] = l_sum;
    asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
    float l_tot = 0.f;
    if constexpr (C::L_IN_MMA) {
      uint32_t lv16[16];
      tmem_ld16(lane_addr + C::TMEM_O + HD + (RV / 16) * 16, lv16);   // column HD + RV sits at index RV % 16 of its chunk
      tmem_wait_ld();
      l_tot = __uint_as_float(lv16[RV % 16]);
    } else {
#pragma unroll
      for (int q2 = 0; q2 < NP; ++q2) l_tot += xch[q2 * 128 + row];
    }
    const float inv = 1.f / l_tot;
    float u[RV > 0 ? RV : 1];
    if constexpr (RV > 0) {
      uint32_t uv[16];
#pragma unroll
      for (int c = 0; c < (RV + 15) / 16; ++c) {
        tmem_ld16(lane_addr + C::TMEM_O + HD + c * 16, uv);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if (c * 16 + k < RV) u[c * 16 + k] = __uint_as_float(uv[k]) * p.s_v;
      }
    }
    __nv_bfloat16* orow = p.out + ((size_t)i_new * p.n_q + (size_t)g * G + hg) * HD;
#pragma unroll 1
    for (int c = part; c < HD / 16; c += NP) {                    // 16-column chunks of this thread
      uint32_t ov[16];
      tmem_ld16(lane_addr + C::TMEM_O + c * 16, ov);
      tmem_wait_ld();
      float o[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) o[k] = __uint_as_float(ov[k]);
      if constexpr (RV > 0) {
#pragma unroll
        for (int jv = 0; jv < RV; ++jv) {
          const uint32_t* bvr = reinterpret_cast<const uint32_t*>(bv_s + (size_t)jv * HD * 2) + c * 8;
          const float uj = u[jv];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t y = bvr[k];
            o[2 * k] += uj * bf16_bits_to_float(y & 0xffff);
            o[2 * k + 1] += uj * bf16_bits_to_float(y >> 16);
          }
        }
      }
      if (row_ok) {
#pragma unroll
        for (int k = 0; k < 16; k += 8) {
          uint4 w;
          w.x = pack_bf16(o[k] * inv, o[k + 1] * inv); w.y = pack_bf16(o[k + 2] * inv, o[k + 3] * inv);
          w.z = pack_bf16(o[k + 4] * inv, o[k + 5] * inv); w.w = pack_bf16(o[k + 6] * inv, o[k + 7] * inv);
          *reinterpret_cast<uint4*>(orow + c * 16 + k) = w;
        }
      }
    }
    }   // NS == 1
  }
  if (NS > 1) {
    // ---- cluster merge of the context splits: block `split` finishes rows [split*R, (split+1)*R) of the tile
    constexpr int XS = C::SPLIT_XS;
    constexpr int NSM = PTC_SOFTMAX_WARPS * 32;
    const int R = (128 + (int)NS - 1) / (int)NS;        // rows per block (the last block may own fewer); 2 <= NS <= 16
    float* xo = reinterpret_cast<float*>(smem);          // the merge area starts at the Q tile: every MMA has completed
    float* xm = xo + 128 * XS;
    float* xl = xm + 128;
    float* mo = xl + 128;                               // merged rows [R][XS]
    float* wts = mo + 64 * XS;                          // [NS][R] weights of the splits
    float* linv = wts + 16 * 64;                        // [R]
    unsigned char* bvs = reinterpret_cast<unsigned char*>(linv + 64);   // B_v[:, g] slice, [RV][HD] bf16
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
    if (warp >= PTC_FIRST_SM_WARP && warp < PTC_FIRST_SM_WARP + PTC_SOFTMAX_WARPS) {
      const int tid = (warp - PTC_FIRST_SM_WARP) * 32 + lane;
      const int r0 = (int)split * R;
      const int nrows = max(0, min(R, 128 - r0));
      auto peer = [&](const float* local, uint32_t s) -> uint32_t {
        uint32_t remote;
        asm("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote) : "r"(smem_u32(local)), "r"(s));
        return remote;
      };
      auto ld1 = [&](uint32_t a) -> float { float v; asm volatile("ld.shared::cluster.f32 %0, [%1];\n" : "=f"(v) : "r"(a)); return v; };
      if constexpr (RV > 0) {
        for (int c = tid; c < RV * (HD / 8); c += NSM) {
          const int j = c / (HD / 8), ch = c % (HD / 8);
          *reinterpret_cast<uint4*>(bvs + (j * HD + ch * 8) * 2) =
              __ldg(reinterpret_cast<const uint4*>(p.B_v + (size_t)j * p.n_kv * HD + (size_t)g * HD + ch * 8));
        }
      }
      if (tid < nrows) {
        float ms[16], M = NEG_BIG, L = 0.f;
#pragma unroll
        for (uint32_t s2 = 0; s2 < 16; ++s2) { ms[s2] = s2 < NS ? ld1(peer(xm + r0 + tid, s2)) : NEG_BIG; M = fmaxf(M, ms[s2]); }
#pragma unroll
        for (uint32_t s2 = 0; s2 < 16; ++s2) {
          if (s2 < NS) {
            const float wv = fast_exp2(ms[s2] - M);
            wts[s2 * R + tid] = wv;
            L += wv * ld1(peer(xl + r0 + tid, s2));               // split order: deterministic
          }
        }
        linv[tid] = L > 0.f ? 1.f / L : 0.f;
      }
      asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
      constexpr int F4 = (HD + RV) / 4;                   // float4 columns of a merged row
      for (int it = tid; it < nrows * F4; it += NSM) {
        const int rl = it / F4, c4 = it % F4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t s2 = 0; s2 < NS; ++s2) {
          const uint32_t a = peer(xo + (r0 + rl) * XS + c4 * 4, s2);
          float4 x;
          asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(a));
          const float wv = wts[s2 * R + rl];
          acc.x += wv * x.x; acc.y += wv * x.y; acc.z += wv * x.z; acc.w += wv * x.w;
        }
        *reinterpret_cast<float4*>(mo + rl * XS + c4 * 4) = acc;
      }
      asm volatile("bar.sync 1, %0;\n" ::"r"(NSM) : "memory");
      // out = (O + s_v U B_v) / l for my rows, eight columns per item
      for (int it = tid; it < nrows * (HD / 8); it += NSM) {
        const int rl = it / (HD / 8), c8 = (it % (HD / 8)) * 8;
        const int rowg = r0 + rl;
        if (rowg >= n_tok * G) continue;
        float o[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] = mo[rl * XS + c8 + k];
        if constexpr (RV > 0) {
#pragma unroll 4
          for (int jv = 0; jv < RV; ++jv) {
            const float uj = mo[rl * XS + HD + jv] * p.s_v;
            const uint4 y = *reinterpret_cast<const uint4*>(bvs + (jv * HD + c8) * 2);
            const uint32_t ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              o[2 * k] += uj * bf16_bits_to_float(ys[k] & 0xffff);
              o[2 * k + 1] += uj * bf16_bits_to_float(ys[k] >> 16);
            }
          }
        }
        const float inv = linv[rl];
        const int i_new = tok0 + rowg / G, hg = rowg % G;
        uint4 w;
        w.x = pack_bf16(o[0] * inv, o[1] * inv); w.y = pack_bf16(o[2] * inv, o[3] * inv);
        w.z = pack_bf16(o[4] * inv, o[5] * inv); w.w = pack_bf16(o[6] * inv, o[7] * inv);
        *reinterpret_cast<uint4*>(p.out + ((size_t)i_new * p.n_q + (size_t)g * G + hg) * HD + c8) = w;
      }
    }
    // nobody leaves while a peer may still read its partial
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  }
  if constexpr (worklist) {
    // end of a piece: nothing of it is in flight any more once every warp is here
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }
  }   // pieces of the work list (one pass in a classic launch)
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace precc
