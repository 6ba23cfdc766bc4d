// LR-reconstructed decode attention (split-KV).
//
// For request b (agent a), kv head g and its G <= 8 query heads the kernels evaluate plain softmax
// attention with K_a = K_base + s_k L^K_a B^K_a and V_a = V_base + s_v L^V_a B^V_a (Eq. 1) without
// building K_a or V_a: the key-side adapter is folded into r extra query coordinates
// (q~ = s_k q B^K_{a,g}^T, contraction length head_dim + r_k) and the value-side adapter into r extra
// output coordinates (U = P L^V_a, then out += s_v U B^V_{a,g}).
//
// Rotary variant (ROPE = true, Appendix D.2): the base cache holds rotated keys, the LR-K rows are not
// rotated, and a rotated key cannot take the fold because the rotation sits between L^K and q.  Per
// page the warp expands E = L^K B^K_{a,g} on the tensor cores (16 x hd), rotates E by the tokens'
// positions (token t of a request sits at position t; rotate-half pairing (c, c + hd/2)), and adds
// s_k E to the key fragments before the score MMA; nothing of K_a is written anywhere.  The value side
// is unchanged.
//
// Streaming core (decode_stream_block): a thread block owns consecutive 16-token pages of one (b, g);
// its warps take pages round-robin, each with a private cp.async ring (no block-wide barrier inside
// the stream loop).  Tokens sit on the MMA M axis:
//   S^T[16 tok x 8 q]   = K'[16 x (hd+r_k)] . Q'^T          (mma.sync m16n8k16, bf16 -> fp32)
//   O^T[(hd+r_v) x 8 q] += V'^T[(hd+r_v) x 16 tok] . P^T     (P^T obtained with movmatrix)
// so no MMA row is wasted on padding.  The block's result (m, l, O') is left in shared memory.
//
// Two ways to combine the blocks of one (b, g):
//   cluster kernel  the splits of a (b, g) form one thread-block cluster (up to 16 blocks); every block sends
//                   the merged values of each output column to the block that owns the column (st.async into
//                   the owner's shared memory, counted on the owner's mbarrier), and the owner adds what it
//                   receives in rank order.  No global scratch, no atomics: the short-latency path for small
//                   batches.
//   ticket kernel   blocks publish their result to a global workspace; the last block to finish a
//                   (b, g) (atomic ticket) merges the records in split order.  Any number of splits.
// The ticket path never waits on another block.  In the cluster path a block waits (bounded, on its own
// mbarrier) for the sends of blocks that are co-scheduled with it by the hardware.
#pragma once
#include "common.cuh"

namespace precc {

struct DecodeParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int32_t* agent_id;
  const int32_t* ctx_len;
  const int32_t* block_table;
  const int32_t* first_block;
  const __nv_bfloat16* k_base;
  const __nv_bfloat16* v_base;
  const __nv_bfloat16* lr_k;
  const __nv_bfloat16* lr_v;
  const __nv_bfloat16* B_k;
  const __nv_bfloat16* B_v;
  float* part;        // ticket kernel: [B][n_kv][max_splits][PART_STRIDE]
  int32_t* tickets;   // ticket kernel: [B][n_kv], zero between calls
  float* raw;         // partial-output mode (ticket kernel): [B][n_kv][PART_STRIDE] records instead of `out`, or null
  uint32_t* status;
  unsigned long long* trace;   // optional [blocks][16] phase timestamps (ns), or null
  const float4* rope;          // rotary variant: [max_pos][hd/4] of (cos c, sin c, cos c+1, sin c+1), c even
  int max_pos;                 // rows of `rope`; a context longer than this raises BAD_INDEX
  int bk_off;                  // rotary variant: byte offset of the B_k slice in dynamic shared memory
  int64_t n_blocks;
  int table_stride;
  int n_q, n_kv, group, n_agents;
  int chunk_tiles, max_splits, stages;
  int pre_stages;              // ring slots a warp fills before it waits for the preceding kernel (the rest follow the wait)
  int max_ctx;                 // the host's bound on ctx_len[b]: it sized the grid, the split and the block table
  float scale_log2, s_k, s_v;
};

constexpr int DEC_WARPS = 4;            // ticket kernel
constexpr int DEC_MAX_SPLITS = 512;
constexpr int DEC_MAX_CLUSTER = 16;
// Overlap with the preceding kernel (programmatic dependent launch): before the kernel waits for its
// predecessor it already reads the index arrays, the adapter matrices and every cache page that holds
// none of the request's last DEC_PDL_TAIL tokens.  The newest tokens (the in-turn append of the preceding
// few-row projection), q and every store stay behind the wait.
constexpr int DEC_PDL_TAIL = 64;

template <int HD, int RK, int RV>
struct DecodeCfg {
  static constexpr int KV_BYTES = PAGE * HD * 2;
  static constexpr int LK_BYTES = PAGE * RK * 2;
  static constexpr int LV_BYTES = PAGE * RV * 2;
  static constexpr int STAGE_BYTES = 2 * KV_BYTES + LK_BYTES + LV_BYTES;
  static constexpr int OW = HD + RV;                 // accumulated output width
  static constexpr int PART_STRIDE = 8 * OW + 16;     // floats: m[8], l[8], O'[8][OW]
  static constexpr int BK_ROWS = RK > 16 ? RK : 16;   // rotary variant: B_k[a][:, g] slice, rows padded to 16
  static constexpr int BK_BYTES = BK_ROWS * HD * 2;
  // shared memory of a block with `warps` warps and `stages` ring slots per warp
  __host__ __device__ static constexpr int ring_bytes(int warps, int stages) { return warps * stages * STAGE_BYTES; }
  static constexpr int OWP = OW + 4;                  // padded head stride of a warp's record in the block merge (OW % 8 == 0)
  static constexpr int WREC = 8 * OWP + 16;           // floats per warp record: m[8], l[8], O'[8 heads][OWP]
  __host__ __device__ static constexpr int merge_bytes(int warps) { return warps * WREC * 4; }
  __host__ __device__ static constexpr int ticket_smem(int stages) {
    int a = ring_bytes(DEC_WARPS, stages), b = merge_bytes(DEC_WARPS);
    int c = (16 + 8 * OW + 16 * DEC_MAX_SPLITS + DEC_WARPS * 8 * OW) * 4 + RV * HD * 2;   // final merge without staging
    int m = a > b ? a : b;
    return (m > c ? m : c) + 64;
  }
  // Cluster kernel.  Behind the ring region sits the receive area that the peers fill with st.async:
  // [CS sources][G heads][cols columns] merged values, then [CS][G] pairs (m, l), then two mbarriers (received
  // bytes; arrival of the B_v slice).  With cols = ceil(W / CS), W <= OW columns and G <= 8:
  // CS G cols + 2 G CS + 1 <= 8 OW + 24 CS floats.
  static constexpr int RECV_FLOATS = 8 * OW + 24 * DEC_MAX_CLUSTER;
  static constexpr int RECV_BYTES = RECV_FLOATS * 4 + 16;
  // Value-side adapter term s_v U B_v.  WEXP: every warp adds it to its own partial on the tensor cores right
  // after its last page (O^T += B_v^T (s_v U)^T: B_v[a][:, g] is staged like a value page of max(r_v, 16) "tokens"
  // behind the receive area).  That takes r_v x hd x 2 bytes more per block; where two blocks of the smallest
  // kind would no longer fit on an SM (head_dim 128 with rank 64) the term is added after the block merge
  // instead, from a copy of B_v that is placed in the ring region once the stream is over.
  static constexpr int BVP = RV > 16 ? RV : 16;
  static constexpr bool WEXP = RV > 0 && ring_bytes(4, 2) + RECV_BYTES + 128 + BVP * HD * 2 + 64 <= 232448 / 2 - 1024;
  static constexpr int BVS_BYTES = WEXP ? BVP * HD * 2 : 0;
  __host__ __device__ static constexpr int cluster_tail(int warps) { return merge_bytes(warps) + (WEXP ? 0 : RV * HD * 2 + 8 * RV * 4); }
  __host__ __device__ static constexpr int cluster_core(int warps, int stages) {   // offset of the receive area
    int a = ring_bytes(warps, stages), b = cluster_tail(warps);
    return ((a > b ? a : b) + 15) / 16 * 16;
  }
  __host__ __device__ static constexpr int cluster_bv(int warps, int stages) {     // offset of the staged B_v slice (WEXP)
    return (cluster_core(warps, stages) + RECV_BYTES + 127) / 128 * 128;
  }
  __host__ __device__ static constexpr int cluster_smem(int warps, int stages) { return cluster_bv(warps, stages) + BVS_BYTES + 64; }
};

struct DecodeTrace {
  unsigned long long* buf;
  __device__ __forceinline__ void operator()(int k) const {
    if (buf && threadIdx.x == 0) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      buf[k] = t;
    }
  }
  // slot 15: the SM the block runs on (placement of co-resident launches)
  __device__ __forceinline__ void where() const {
    if (buf && threadIdx.x == 0) {
      unsigned int id;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(id));
      buf[15] = id;
    }
  }
};

// Query fragments of one (b, g): B operand of the score MMA (k = head-dim coordinate, n = query head).
template <int HD>
__device__ __forceinline__ void load_q_frags(const DecodeParams& p, int b, int g, uint32_t (&qb)[HD / 16][2]) {
  const int lane = threadIdx.x & 31;
  const int qrow = lane >> 2, qk = (lane & 3) * 2;
  const __nv_bfloat16* qsrc = p.q + ((size_t)b * p.n_q + (size_t)g * p.group + qrow) * HD;
#pragma unroll
  for (int kc = 0; kc < HD / 16; ++kc) {
    if (qrow < p.group) {
      qb[kc][0] = __ldg(reinterpret_cast<const uint32_t*>(qsrc + kc * 16 + qk));
      qb[kc][1] = __ldg(reinterpret_cast<const uint32_t*>(qsrc + kc * 16 + 8 + qk));
    } else {
      qb[kc][0] = 0u; qb[kc][1] = 0u;
    }
  }
}

// Streams pages [tile0, tile_end) of (b, g) through the NW warps of the block and leaves the block's
// result in shared memory as floats  res = [ m[8] | l[8] | O'[G][OW] ]  at the start of `smem`
// (m = running maximum in the log2 domain, l = softmax denominator, O' = unnormalised output with the
// r_v LR-V coordinates appended).  Ends with a __syncthreads().  A block with no pages yields
// m = NEG_BIG, l = 0, O' = 0.  With MERGE = false it stops one step earlier: the warps' records
// [warp][ m[8] | l[8] | O'[8][OWP] ] are written to the start of `smem`, no barrier follows.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory"); }

// B_v slice staged in shared memory for the warps' own adapter term (cluster kernel): `bar` completes when
// every thread's copies have landed.
struct WarpExpand {
  bool on;
  uint32_t bv_u32, bar;
};

template <int HD, int RK, int RV, int NW, bool ROPE, bool MERGE = true>
__device__ __forceinline__ void decode_stream_block(const DecodeParams& p, unsigned char* smem, int b, int g, int ctx,
                                                    int agent, bool use_lr, int tile0, int tile_end, const DecodeTrace& mark,
                                                    const WarpExpand wexp = WarpExpand{false, 0u, 0u}) {
  static_assert(!ROPE || RK > 0, "the rotary variant only differs when there is a key-side adapter");
  using C = DecodeCfg<HD, RK, RV>;
  constexpr int OW = C::OW;
  constexpr int KC = HD / 16;                         // k-chunks of the base part
  constexpr int KX = (RK + 15) / 16;                  // k-chunks of the LR-K part
  constexpr int MT = HD / 16;                         // m-tiles of the base output
  constexpr int MX = (RV + 15) / 16;                  // m-tiles of the LR-V output
  constexpr int CPR_KV = HD / 8;
  constexpr int CPR_LK = RK > 0 ? RK / 8 : 1;
  constexpr int CPR_LV = RV > 0 ? RV / 8 : 1;
  constexpr int NT = NW * 32;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.group;
  const int qk = (lane & 3) * 2;
  // this warp's pages: tile0 + warp + NW * i
  const int my_n = (tile_end - tile0 - warp + NW - 1) / NW;   // may be <= 0
  const uint32_t ring_u32 = smem_u32(smem + (size_t)warp * p.stages * C::STAGE_BYTES);

  // ---- physical block ids, fetched 32 pages at a time, one batch ahead
  auto load_phys = [&](int batch) -> int {
    const int i = batch * 32 + lane;
    if (i >= my_n) return 0;
    const int t = tile0 + warp + NW * i;
    int ph = p.block_table ? __ldg(p.block_table + (size_t)b * p.table_stride + t)
                           : (p.first_block ? __ldg(p.first_block + b) : 0) + t;
    if (ph < 0 || ph >= p.n_blocks) { atomicOr(p.status, StatusBits::BAD_INDEX); ph = 0; }
    return ph;
  };
  int phys_cur = load_phys(0);
  int phys_nxt = load_phys(1);

  const __nv_bfloat16* lrk_a = RK > 0 ? p.lr_k + (size_t)agent * p.n_blocks * PAGE * RK : nullptr;
  const __nv_bfloat16* lrv_a = RV > 0 ? p.lr_v + (size_t)agent * p.n_blocks * PAGE * RV : nullptr;

  // ---- page copies.  Everything that does not change from page to page is computed once: lane l moves the
  //      16-byte chunks l + 32 j of each tile; the source of chunk j is (page base + 16 l) + 512 j, its swizzled
  //      destination repeats with the period of (row & 7), so two (or four) offsets cover all j.  Per page that
  //      leaves one 64-bit multiply-add per cache array and one cp.async per chunk.
  constexpr int KV_PER_LANE = PAGE * CPR_KV / 32;        // 4 (head_dim 64) or 8 (128)
  constexpr int KV_PERIOD = CPR_KV / 4;                  // 2 or 4: rows advance by 32 / CPR_KV per j, the swizzle by row & 7
  uint32_t kv_dst[KV_PERIOD];
#pragma unroll
  for (int jj = 0; jj < KV_PERIOD; ++jj) {
    const int c = lane + 32 * jj;
    kv_dst[jj] = swz_off<CPR_KV>(c / CPR_KV, c % CPR_KV);
  }
  const int kv_row0 = lane / CPR_KV;                     // row of chunk j: kv_row0 + j * (32 / CPR_KV)
  constexpr int LK_PER_LANE = RK > 0 ? (PAGE * CPR_LK + 31) / 32 : 0;   // 1, 1, 2, 4 for rank 8, 16, 32, 64
  constexpr int LV_PER_LANE = RV > 0 ? (PAGE * CPR_LV + 31) / 32 : 0;
  constexpr int LK_PERIOD = CPR_LK >= 8 ? 2 : 1, LV_PERIOD = CPR_LV >= 8 ? 2 : 1;
  uint32_t lk_dst[LK_PERIOD], lv_dst[LV_PERIOD];
#pragma unroll
  for (int jj = 0; jj < LK_PERIOD; ++jj) { const int c = lane + 32 * jj; lk_dst[jj] = swz_off<CPR_LK>(c / CPR_LK, c % CPR_LK); }
#pragma unroll
  for (int jj = 0; jj < LV_PERIOD; ++jj) { const int c = lane + 32 * jj; lv_dst[jj] = swz_off<CPR_LV>(c / CPR_LV, c % CPR_LV); }
  const bool lr_lane_k = RK > 0 && use_lr && lane < PAGE * CPR_LK;     // rank 8: 16 chunks, lanes 0..15 only
  const bool lr_lane_v = RV > 0 && use_lr && lane < PAGE * CPR_LV;
  const int lv_row0 = lane / CPR_LV;
  const unsigned char* const k_lane = reinterpret_cast<const unsigned char*>(p.k_base) + (size_t)g * C::KV_BYTES + lane * 16;
  const ptrdiff_t v_minus_k = reinterpret_cast<const unsigned char*>(p.v_base) - reinterpret_cast<const unsigned char*>(p.k_base);
  const unsigned char* const lk_lane = reinterpret_cast<const unsigned char*>(lrk_a) + lane * 16;
  const unsigned char* const lv_lane = reinterpret_cast<const unsigned char*>(lrv_a) + lane * 16;
  const size_t kv_block_bytes = (size_t)p.n_kv * C::KV_BYTES;
  int issue_slot = 0;                                   // ring slot of the next page to request: i % stages, kept incrementally

  auto issue_tile = [&](int i) {
    if (i < my_n) {
      if ((i & 31) == 0 && i > 0) { phys_cur = phys_nxt; phys_nxt = load_phys((i >> 5) + 1); }
      const int ph = __shfl_sync(0xffffffffu, phys_cur, i & 31);
      const int t = tile0 + warp + NW * i;
      const int valid = ctx - t * PAGE;                 // >= PAGE for every page but the request's last one
      const uint32_t st = ring_u32 + (uint32_t)issue_slot * C::STAGE_BYTES;
      const unsigned char* ksrc = k_lane + (size_t)ph * kv_block_bytes;
      const unsigned char* vsrc = ksrc + v_minus_k;
      if (valid >= PAGE) {
#pragma unroll
        for (int j = 0; j < KV_PER_LANE; ++j) {
          const uint32_t dst = st + kv_dst[j % KV_PERIOD] + (j / KV_PERIOD) * (KV_PERIOD * 512);
          cp_async16(dst, ksrc + j * 512, 16);
          cp_async16(dst + C::KV_BYTES, vsrc + j * 512, 16);
        }
        if (lr_lane_k) {
          const unsigned char* src = lk_lane + (size_t)ph * C::LK_BYTES;
#pragma unroll
          for (int j = 0; j < LK_PER_LANE; ++j)
            cp_async16(st + 2 * C::KV_BYTES + lk_dst[j % LK_PERIOD] + (j / LK_PERIOD) * (LK_PERIOD * 512), src + j * 512, 16);
        }
        if (lr_lane_v) {
          const unsigned char* src = lv_lane + (size_t)ph * C::LV_BYTES;
#pragma unroll
          for (int j = 0; j < LV_PER_LANE; ++j)
            cp_async16(st + 2 * C::KV_BYTES + C::LK_BYTES + lv_dst[j % LV_PERIOD] + (j / LV_PERIOD) * (LV_PERIOD * 512), src + j * 512, 16);
        }
      } else {
        // the request's last, partial page: value rows past the context are zero-filled - their weight is zero,
        // but 0 * garbage (an unwritten slot may hold NaN) must not reach the accumulators
#pragma unroll
        for (int j = 0; j < KV_PER_LANE; ++j) {
          const uint32_t dst = st + kv_dst[j % KV_PERIOD] + (j / KV_PERIOD) * (KV_PERIOD * 512);
          cp_async16(dst, ksrc + j * 512, 16);
          cp_async16(dst + C::KV_BYTES, vsrc + j * 512, kv_row0 + j * (32 / CPR_KV) < valid ? 16 : 0);
        }
        if (lr_lane_k) {
          const unsigned char* src = lk_lane + (size_t)ph * C::LK_BYTES;
#pragma unroll
          for (int j = 0; j < LK_PER_LANE; ++j)
            cp_async16(st + 2 * C::KV_BYTES + lk_dst[j % LK_PERIOD] + (j / LK_PERIOD) * (LK_PERIOD * 512), src + j * 512, 16);
        }
        if (lr_lane_v) {
          const unsigned char* src = lv_lane + (size_t)ph * C::LV_BYTES;
#pragma unroll
          for (int j = 0; j < LV_PER_LANE; ++j)
            cp_async16(st + 2 * C::KV_BYTES + C::LK_BYTES + lv_dst[j % LV_PERIOD] + (j / LV_PERIOD) * (LV_PERIOD * 512), src + j * 512,
                       lv_row0 + j * (32 / CPR_LV) < valid ? 16 : 0);
        }
      }
    }
    if (++issue_slot == p.stages) issue_slot = 0;
    cp_async_commit();
  };

  // ---- B_k fragments for the query fold are requested first (a few small loads), so that they do
  //      not queue behind the page stream; large ranks would need too many registers and load later
  constexpr bool PRELOAD_BK = !ROPE && RK > 0 && KX * KC * 4 <= 32;
  const __nv_bfloat16* Bk = RK > 0 ? p.B_k + ((size_t)agent * RK) * ((size_t)p.n_kv * HD) + (size_t)g * HD : nullptr;
  const size_t bk_rs = (size_t)p.n_kv * HD;     // row stride of B_k
  auto load_bk = [&](int jt, int kc, uint32_t (&a)[4]) {
    const __nv_bfloat16* r0 = Bk + (size_t)(jt * 16 + (lane >> 2)) * bk_rs + qk + kc * 16;
    a[0] = __ldg(reinterpret_cast<const uint32_t*>(r0));
    a[2] = __ldg(reinterpret_cast<const uint32_t*>(r0 + 8));
    if (RK >= 16) {
      a[1] = __ldg(reinterpret_cast<const uint32_t*>(r0 + 8 * bk_rs));
      a[3] = __ldg(reinterpret_cast<const uint32_t*>(r0 + 8 * bk_rs + 8));
    } else {
      a[1] = 0u; a[3] = 0u;
    }
  };
  // Small ranks: every warp holds the B_k fragments itself (requested here, before the wait for the preceding
  // kernel) and folds on its own, so that nothing but the arrival of q stands between the wait and the first
  // score MMA.  Large ranks: only warp 0 loads B_k (at the fold, the fragments do not fit in registers) and the
  // other warps pick the folded fragments up from shared memory.
  uint32_t bk_pre[PRELOAD_BK ? KX * KC : 1][4];
  if constexpr (PRELOAD_BK) {
    if (use_lr) {
#pragma unroll
      for (int jt = 0; jt < KX; ++jt)
#pragma unroll
        for (int kc = 0; kc < KC; ++kc) load_bk(jt, kc, bk_pre[jt * KC + kc]);
    }
  }
  // ---- rotary variant: the B_k[a][:, g] slice goes to shared memory ([BK_ROWS][HD], swizzled like a
  //      key page; rows >= RK are zero); requested before the page stream, stored after it is issued
  constexpr int BK_CHUNKS = ROPE ? C::BK_ROWS * CPR_KV : 0;
  constexpr int BK_PER_THREAD = ROPE ? (BK_CHUNKS + NT - 1) / NT : 1;
  uint4 bk_stage[BK_PER_THREAD];
  if constexpr (ROPE) {
#pragma unroll
    for (int k = 0; k < BK_PER_THREAD; ++k) {
      const int c = threadIdx.x + k * NT;
      const int j = c / CPR_KV, ch = c % CPR_KV;
      bk_stage[k] = (c < BK_CHUNKS && j < RK && use_lr) ? __ldg(reinterpret_cast<const uint4*>(Bk + (size_t)j * bk_rs + ch * 8))
                                                        : make_uint4(0u, 0u, 0u, 0u);
    }
  }
  // the LoRA scale is folded into the slice (one bf16 rounding of s_k B; exact for power-of-two scales)
  auto scale2 = [&](uint32_t v) -> uint32_t {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v));
    return pack_bf16(f.x * p.s_k, f.y * p.s_k);
  };
  // ---- start the stream: every ring slot is filled at once.  Pages that cannot hold one of the request's
  //      last DEC_PDL_TAIL tokens are requested while the preceding kernel may still be running; the wait
  //      for that kernel comes next, and the pages it may have appended to are requested after it.
  const int safe_tiles = max(0, ctx - DEC_PDL_TAIL) / PAGE;
  // Cluster schedule: the last warp is the block's scout.  It requests only its first page before the wait, so
  // that in a block that starts when its predecessor is already over - where filling the rings is throttled by
  // the SM's limit on requests in flight and takes two DRAM round trips - the q lines are requested about one
  // round trip earlier; the other warps' q loads then hit in L1.  A block that starts early has time to spare.
  const bool scout = !MERGE && warp == NW - 1;
  // q is the predecessor's to write, so it is read after the wait - but its lines can be brought into L2 now (L2 is
  // the point of coherence: a later write by the predecessor lands there too), which turns the one load that stands
  // between the wait and the first MMA from a DRAM round trip into an L2 hit
  if (warp == NW - 1 && lane * 128 < G * HD * 2)
    asm volatile("prefetch.global.L2 [%0];\n" ::"l"(reinterpret_cast<const unsigned char*>(p.q + ((size_t)b * p.n_q + (size_t)g * G) * HD) + lane * 128));
  const int pre_cap = scout ? 1 : p.pre_stages;
  int n_pre = 0;
  for (; n_pre < pre_cap; ++n_pre) {
    if (n_pre < my_n && tile0 + warp + NW * n_pre >= safe_tiles) break;
    issue_tile(n_pre);
  }
  // Cluster schedule: the pages that will be requested as soon as the first ring slots are free are brought into L2
  // now (a hint, not a read: L2 is the point of coherence, so this is allowed ahead of the wait for any page), which
  // turns the round trip that a shallow ring exposes in the loop from a DRAM access into an L2 hit.  Only for short
  // streams (at most two ring generations per warp), which are bound by that latency; a longer stream hides it behind
  // its ring, and the extra requests cost it 2 .. 6 % (measured at head_dim 128, 8192 .. 131072 tokens).
  if (!MERGE && my_n <= 2 * p.stages) {
    constexpr int KV_LINES = C::KV_BYTES / 128;
    const unsigned char* kb = reinterpret_cast<const unsigned char*>(p.k_base) + (size_t)g * C::KV_BYTES;
    for (int i = p.stages; i < my_n && i < 2 * p.stages && i < 32; ++i) {
      const int ph = __shfl_sync(0xffffffffu, phys_cur, i);
      const unsigned char* ksrc = kb + (size_t)ph * kv_block_bytes;
      for (int l = lane; l < 2 * KV_LINES; l += 32) {
        const unsigned char* a = l < KV_LINES ? ksrc + l * 128 : ksrc + v_minus_k + (l - KV_LINES) * 128;
        asm volatile("prefetch.global.L2 [%0];\n" ::"l"(a));
      }
      if (use_lr) {
        if (RK > 0 && lane * 128 < C::LK_BYTES)
          asm volatile("prefetch.global.L2 [%0];\n" ::"l"(reinterpret_cast<const unsigned char*>(lrk_a) + (size_t)ph * C::LK_BYTES + lane * 128));
        if (RV > 0 && lane * 128 < C::LV_BYTES)
          asm volatile("prefetch.global.L2 [%0];\n" ::"l"(reinterpret_cast<const unsigned char*>(lrv_a) + (size_t)ph * C::LV_BYTES + lane * 128));
      }
    }
  }
  mark(8);
  pdl_wait();                 // the predecessor has completed: its q, its cache rows and its workspace are visible
  mark(9);
  pdl_launch_dependents();
  uint32_t qb[HD / 16][2];
  load_q_frags<HD>(p, b, g, qb);
  for (int i = n_pre; i < p.stages; ++i) issue_tile(i);
  mark(2);
  const uint32_t bk_u32 = smem_u32(smem + p.bk_off);
  if constexpr (ROPE) {
#pragma unroll
    for (int k = 0; k < BK_PER_THREAD; ++k) {
      const int c = threadIdx.x + k * NT;
      if (c < BK_CHUNKS)
        *reinterpret_cast<uint4*>(smem + p.bk_off + swz_off<CPR_KV>(c / CPR_KV, c % CPR_KV)) =
            make_uint4(scale2(bk_stage[k].x), scale2(bk_stage[k].y), scale2(bk_stage[k].z), scale2(bk_stage[k].w));
    }
    __syncthreads();
  }

  // ---- folded key-side adapter q~ = s_k q B_k[a][:, g]^T, computed on the tensor cores as
  //      q~^T[j x q] = B_k[j x c] . q^T[c x q]; the accumulator fragment, transposed with movmatrix,
  //      is exactly the B operand (k = j, n = query) needed by the score MMA.
  uint32_t qxb[KX > 0 ? KX : 1][2];
  if constexpr (RK > 0 && !ROPE) {
    __shared__ uint32_t qx_share[KX > 0 ? KX : 1][2][32];
#pragma unroll
    for (int jt = 0; jt < KX; ++jt) { qxb[jt][0] = 0u; qxb[jt][1] = 0u; }
    if ((PRELOAD_BK || warp == 0) && use_lr) {
#pragma unroll
      for (int jt = 0; jt < KX; ++jt) {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kc = 0; kc < KC; ++kc) {
          if constexpr (PRELOAD_BK) {
            mma_bf16_16816(c, bk_pre[jt * KC + kc], qb[kc][0], qb[kc][1]);
          } else {
            uint32_t a[4];
            load_bk(jt, kc, a);
            mma_bf16_16816(c, a, qb[kc][0], qb[kc][1]);
          }
        }
        qxb[jt][0] = movmatrix_t(pack_bf16(c[0] * p.s_k, c[1] * p.s_k));
        qxb[jt][1] = movmatrix_t(pack_bf16(c[2] * p.s_k, c[3] * p.s_k));
        if constexpr (!PRELOAD_BK) {
          qx_share[jt][0][lane] = qxb[jt][0];
          qx_share[jt][1][lane] = qxb[jt][1];
        }
      }
    }
    if constexpr (!PRELOAD_BK) {
      __syncthreads();
      if (warp != 0 && use_lr) {
#pragma unroll
        for (int jt = 0; jt < KX; ++jt) { qxb[jt][0] = qx_share[jt][0][lane]; qxb[jt][1] = qx_share[jt][1][lane]; }
      }
    }
  }

  // ---- online-softmax state: this lane's two query columns (2*(lane&3), +1)
  float m0 = NEG_BIG, m1 = NEG_BIG, l0 = 0.f, l1 = 0.f;
  float o[MT + MX][4];
#pragma unroll
  for (int i = 0; i < MT + MX; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8;   // K' A-operand: row, chunk parity
  const int a_cpar = lane >> 4;
  const int v_row = (lane & 7) + (lane >> 4) * 8;         // V'^T A-operand (transposed load)
  const int v_cpar = (lane >> 3) & 1;

  // ---- rotary variant: (cos, sin) of this lane's tokens (rows lane>>2 and +8 of the page) and columns
  //      (n-tiles 2kc and 2kc+1 of the lower half), fetched one page ahead
  constexpr int KH = KC / 2;
  constexpr bool CS_AHEAD = true;                      // wider heads: the table entries are loaded at their use
  float4 cs[ROPE && CS_AHEAD ? KH : 1][2][2];           // [chunk pair][n-tile][row]
  auto load_cs = [&](int i) {
    if constexpr (ROPE && CS_AHEAD) {
      if (i < my_n && use_lr) {
        const int t = tile0 + warp + NW * i;
        const int pos0 = min(t * PAGE + (lane >> 2), p.max_pos - 1), pos1 = min(t * PAGE + (lane >> 2) + 8, p.max_pos - 1);
#pragma unroll
        for (int kc = 0; kc < KH; ++kc)
#pragma unroll
          for (int n2 = 0; n2 < 2; ++n2) {
            const int c4 = (kc * 16 + n2 * 8 + qk) >> 1;           // float4 index: two columns per entry
            cs[kc][n2][0] = __ldg(p.rope + (size_t)pos0 * (HD / 4) + c4);
            cs[kc][n2][1] = __ldg(p.rope + (size_t)pos1 * (HD / 4) + c4);
          }
      }
    }
  };
  load_cs(0);

  mark(3);
  int use_slot = 0;                    // ring slot of page i: i % stages, kept incrementally
  for (int i = 0; i < my_n; ++i) {
    switch (p.stages) {                // ring depth 2 .. 8: all but the newest (depth - 1) groups have landed
      case 2: cp_async_wait<1>(); break;
      case 3: cp_async_wait<2>(); break;
      case 4: cp_async_wait<3>(); break;
      case 5: cp_async_wait<4>(); break;
      case 6: cp_async_wait<5>(); break;
      case 7: cp_async_wait<6>(); break;
      default: cp_async_wait<7>(); break;
    }
    __syncwarp();                      // page i is visible to all lanes
    if (i == 0) mark(4);
    const uint32_t st = ring_u32 + (uint32_t)use_slot * C::STAGE_BYTES;
    if (++use_slot == p.stages) use_slot = 0;
    const int t = tile0 + warp + NW * i;
    const int valid = ctx - t * PAGE;   // >= 1; tokens >= valid are masked

    float s[4] = {0.f, 0.f, 0.f, 0.f};
    if (ROPE && use_lr) {
      if constexpr (ROPE) {
        // L^K fragments of the page (A operand of the expansion), all rank chunks
        uint32_t la[KX][4];
#pragma unroll
        for (int jx = 0; jx < KX; ++jx) {
          if constexpr (RK >= 16) {
            ldsm_x4(la[jx], st + 2 * C::KV_BYTES + swz_off<CPR_LK>(a_row, 2 * jx + a_cpar));
          } else {
            la[jx][2] = 0u; la[jx][3] = 0u;
            ldsm_x2(la[jx][0], la[jx][1], st + 2 * C::KV_BYTES + swz_off<1>(a_row, 0));
          }
        }
#pragma unroll
        for (int kc = 0; kc < KH; ++kc) {
          // E for columns [16kc, 16kc+16) and their rotation partners [16kc + hd/2, ...)
          float e[2][2][4];                              // [half][n-tile][c]
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
            for (int n2 = 0; n2 < 2; ++n2) { e[hf][n2][0] = e[hf][n2][1] = e[hf][n2][2] = e[hf][n2][3] = 0.f; }
#pragma unroll
            for (int jx = 0; jx < KX; ++jx) {
              uint32_t bf[4];
              ldsm_x4_t(bf, bk_u32 + swz_off<CPR_KV>(16 * jx + a_row, 2 * (kc + hf * KH) + a_cpar));
              mma_bf16_16816(e[hf][0], la[jx], bf[0], bf[1]);
              mma_bf16_16816(e[hf][1], la[jx], bf[2], bf[3]);
            }
          }
          uint32_t alo[4], ahi[4];
          ldsm_x4(alo, st + swz_off<CPR_KV>(a_row, 2 * kc + a_cpar));
          ldsm_x4(ahi, st + swz_off<CPR_KV>(a_row, 2 * (kc + KH) + a_cpar));
          float4 csl[2][2];
          if constexpr (!CS_AHEAD) {
            const int pos0 = min(t * PAGE + (lane >> 2), p.max_pos - 1), pos1 = min(t * PAGE + (lane >> 2) + 8, p.max_pos - 1);
#pragma unroll
            for (int n2 = 0; n2 < 2; ++n2) {
              const int c4i = (kc * 16 + n2 * 8 + qk) >> 1;
              csl[n2][0] = __ldg(p.rope + (size_t)pos0 * (HD / 4) + c4i);
              csl[n2][1] = __ldg(p.rope + (size_t)pos1 * (HD / 4) + c4i);
            }
          }
#pragma unroll
          for (int n2 = 0; n2 < 2; ++n2)
#pragma unroll
            for (int r = 0; r < 2; ++r) {
              const float4 c4 = CS_AHEAD ? cs[CS_AHEAD ? kc : 0][n2][r] : csl[n2][r];   // (cos c, sin c, cos c+1, sin c+1)
              const float lo0 = e[0][n2][2 * r], lo1 = e[0][n2][2 * r + 1];
              const float hi0 = e[1][n2][2 * r], hi1 = e[1][n2][2 * r + 1];
              const uint32_t rl = pack_bf16(lo0 * c4.x - hi0 * c4.y, lo1 * c4.z - hi1 * c4.w);
              const uint32_t rh = pack_bf16(hi0 * c4.x + lo0 * c4.y, hi1 * c4.z + lo1 * c4.w);
              const int f = n2 * 2 + r;                  // A fragment register: (n-tile, row half)
              // packed bf16 add: the rotated rank-r term is rounded to bf16 once before it joins the key
              *reinterpret_cast<__nv_bfloat162*>(&alo[f]) = __hadd2(*reinterpret_cast<const __nv_bfloat162*>(&alo[f]),
                                                                   *reinterpret_cast<const __nv_bfloat162*>(&rl));
              *reinterpret_cast<__nv_bfloat162*>(&ahi[f]) = __hadd2(*reinterpret_cast<const __nv_bfloat162*>(&ahi[f]),
                                                                   *reinterpret_cast<const __nv_bfloat162*>(&rh));
            }
          mma_bf16_16816(s, alo, qb[kc][0], qb[kc][1]);
          mma_bf16_16816(s, ahi, qb[kc + KH][0], qb[kc + KH][1]);
        }
        load_cs(i + 1);
      }
    } else {
#pragma unroll
      for (int kc = 0; kc < KC; ++kc) {
        uint32_t a[4];
        ldsm_x4(a, st + swz_off<CPR_KV>(a_row, 2 * kc + a_cpar));
        mma_bf16_16816(s, a, qb[kc][0], qb[kc][1]);
      }
    }
    if (!use_lr || ROPE) {
    } else if constexpr (RK >= 16) {
#pragma unroll
      for (int kc = 0; kc < KX; ++kc) {
        uint32_t a[4];
        ldsm_x4(a, st + 2 * C::KV_BYTES + swz_off<CPR_LK>(a_row, 2 * kc + a_cpar));
        mma_bf16_16816(s, a, qxb[kc][0], qxb[kc][1]);
      }
    } else if constexpr (RK == 8) {
      uint32_t a[4] = {0u, 0u, 0u, 0u};
      ldsm_x2(a[0], a[1], st + 2 * C::KV_BYTES + swz_off<1>(a_row, 0));
      mma_bf16_16816(s, a, qxb[0][0], 0u);
    }

    // softmax over the token axis (rows of S^T): rows lane>>2 and (lane>>2)+8
    const int tok0 = lane >> 2;
    float z0 = s[0] * p.scale_log2, z1 = s[1] * p.scale_log2, z2 = s[2] * p.scale_log2, z3 = s[3] * p.scale_log2;
    if (tok0 >= valid) { z0 = -INFINITY; z1 = -INFINITY; }
    if (tok0 + 8 >= valid) { z2 = -INFINITY; z3 = -INFINITY; }
    float mx0 = fmaxf(z0, z2), mx1 = fmaxf(z1, z3);
#pragma unroll
    for (int d = 4; d <= 16; d <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, d));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, d));
    }
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);
    const float p0 = fast_exp2(z0 - mn0), p1 = fast_exp2(z1 - mn1);
    const float p2 = fast_exp2(z2 - mn0), p3 = fast_exp2(z3 - mn1);
    l0 = l0 * al0 + p0 + p2;
    l1 = l1 * al1 + p1 + p3;
    m0 = mn0; m1 = mn1;
    const uint32_t pb0 = movmatrix_t(pack_bf16(p0, p1));   // P^T: k = tokens 0..7
    const uint32_t pb1 = movmatrix_t(pack_bf16(p2, p3));   //      k = tokens 8..15
#pragma unroll
    for (int mt = 0; mt < MT + MX; ++mt) { o[mt][0] *= al0; o[mt][1] *= al1; o[mt][2] *= al0; o[mt][3] *= al1; }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      uint32_t a[4];
      ldsm_x4_t(a, st + C::KV_BYTES + swz_off<CPR_KV>(v_row, 2 * mt + v_cpar));
      mma_bf16_16816(o[mt], a, pb0, pb1);
    }
    if (!use_lr) {
    } else if constexpr (RV >= 16) {
#pragma unroll
      for (int mx = 0; mx < MX; ++mx) {
        uint32_t a[4];
        ldsm_x4_t(a, st + 2 * C::KV_BYTES + C::LK_BYTES + swz_off<CPR_LV>(v_row, 2 * mx + v_cpar));
        mma_bf16_16816(o[MT + mx], a, pb0, pb1);
      }
    } else if constexpr (RV == 8) {
      uint32_t a[4] = {0u, 0u, 0u, 0u};
      ldsm_x2_t(a[0], a[2], st + 2 * C::KV_BYTES + C::LK_BYTES + swz_off<1>(a_row, 0));
      mma_bf16_16816(o[MT], a, pb0, pb1);
    }
    __syncwarp();                      // all lanes are done with this slot
    issue_tile(i + p.stages);
  }
  cp_async_wait<0>();
  if constexpr (!MERGE && C::WEXP) {
    // value-side adapter term of this warp's partial, O^T += B_v^T (s_v U)^T: one more "value page" whose tokens
    // are the rank coordinates; U (fp32 accumulators) enters as a bf16 pair hi + lo, i.e. with 16 mantissa bits
    if (wexp.on) {
      mbar_wait(wexp.bar, 0, p.status);
#pragma unroll
      for (int mx = 0; mx < MX; ++mx) {
        const float u0 = o[MT + mx][0] * p.s_v, u1 = o[MT + mx][1] * p.s_v, u2 = o[MT + mx][2] * p.s_v, u3 = o[MT + mx][3] * p.s_v;
        const uint32_t h01 = pack_bf16(u0, u1), h23 = pack_bf16(u2, u3);
        const uint32_t l01 = pack_bf16(u0 - __uint_as_float(h01 << 16), u1 - __uint_as_float(h01 & 0xffff0000u));
        const uint32_t l23 = pack_bf16(u2 - __uint_as_float(h23 << 16), u3 - __uint_as_float(h23 & 0xffff0000u));
        const uint32_t bh0 = movmatrix_t(h01), bh1 = movmatrix_t(h23), bl0 = movmatrix_t(l01), bl1 = movmatrix_t(l23);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          uint32_t a[4];
          ldsm_x4_t(a, wexp.bv_u32 + swz_off<CPR_KV>(16 * mx + v_row, 2 * mt + v_cpar));
          mma_bf16_16816(o[mt], a, bh0, bh1);
          mma_bf16_16816(o[mt], a, bl0, bl1);
        }
      }
    }
  }
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, d);
    l1 += __shfl_xor_sync(0xffffffffu, l1, d);
  }
  mark(5);
  // Cluster schedule: the cluster barrier that every block arrived at when the kernel started (it makes the peers'
  // mbarriers visible) is waited for here, where a warp that is done early waits for the others anyway.
  if constexpr (!MERGE) cluster_wait();

  // ---- merge the warps of this block: smem [warp][ m[8] | l[8] | O'[8 heads][OWP] ], OWP = OW + 4: a store
  //      instruction touches heads cq = 0, 2, 4, 6 (2 OWP = 8 mod 32 banks apart) at rows r = 0..7, i.e. 32 different
  //      banks, and the merging threads load consecutive columns: both free of bank conflicts
  __syncthreads();
  mark(11);
  float* mg = reinterpret_cast<float*>(smem);
  constexpr int OWP = C::OWP;
  constexpr int WREC = C::WREC;
  {
    float* w = mg + warp * WREC;
    if (lane < 4) { w[2 * lane] = m0; w[2 * lane + 1] = m1; w[8 + 2 * lane] = l0; w[8 + 2 * lane + 1] = l1; }
    const int r = lane >> 2, cq = (lane & 3) * 2;
    float* w0 = w + 16 + cq * OWP;         // query head cq, cq + 1
#pragma unroll
    for (int mt = 0; mt < MT + MX; ++mt) {
      if (!MERGE && C::WEXP && mt >= MT && wexp.on) break;      // the LR-V coordinates are spent: nobody reads them
      const int row = mt * 16 + r;
      if (row < OW) { w0[row] = o[mt][0]; w0[OWP + row] = o[mt][1]; }
      if (row + 8 < OW) { w0[row + 8] = o[mt][2]; w0[OWP + row + 8] = o[mt][3]; }
    }
  }
  if constexpr (!MERGE) return;          // the caller merges the warp records itself (after a block barrier of its own)
  __syncthreads();
  mark(13);
  // every thread merges its own elements and derives the warp weights of its query row itself
  // (a few redundant shared-memory reads instead of a serial phase and a barrier); element
  // G*OW + h is the pair (m, l) of row h
  const int n_el = G * OW;
  constexpr int PER_THREAD = (8 * OW + 8 + NT - 1) / NT;
  float acc[PER_THREAD], acc_m[PER_THREAD];
#pragma unroll
  for (int k = 0; k < PER_THREAD; ++k) {
    const int e = threadIdx.x + k * NT;
    float v = 0.f, M = NEG_BIG;
    if (e < n_el + 8) {
      const bool is_ml = e >= n_el;
      const int h = is_ml ? e - n_el : e / OW;
      const int src = is_ml ? 8 + h : 16 + h * OWP + (e % OW);
      float mw[NW], xw[NW];
#pragma unroll
      for (int w = 0; w < NW; ++w) { mw[w] = mg[w * WREC + h]; xw[w] = mg[w * WREC + src]; }
#pragma unroll
      for (int w = 0; w < NW; ++w) M = fmaxf(M, mw[w]);
#pragma unroll
      for (int w = 0; w < NW; ++w) v += xw[w] * fast_exp2(mw[w] - M);   // warp order: deterministic
    }
    acc[k] = v; acc_m[k] = M;
  }
  mark(14);
  __syncthreads();   // all reads of the warp records are done; the region is reused for the result
#pragma unroll
  for (int k = 0; k < PER_THREAD; ++k) {
    const int e = threadIdx.x + k * NT;
    if (e < n_el) mg[16 + e] = acc[k];
    else if (e < n_el + 8) { mg[e - n_el] = acc_m[k]; mg[8 + e - n_el] = acc[k]; }
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// Ticket kernel: grid (split, kv head, request), DEC_WARPS warps.
template <int HD, int RK, int RV, bool ROPE = false>
__global__ void __launch_bounds__(DEC_WARPS * 32)
lr_attend_decode_kernel(const DecodeParams p) {
  using C = DecodeCfg<HD, RK, RV>;
  // partial-output mode has no rotary entry point: compiled out of the rotary instances (which sit at the
  // register limit; the extra branches cost them 14 % through register allocation alone)
  float* const raw_out = ROPE ? nullptr : p.raw;
  constexpr int OW = C::OW;
  constexpr int NT = DEC_WARPS * 32;
  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int G = p.group;
  const int cta_lin = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
  const DecodeTrace mark{p.trace ? p.trace + (size_t)cta_lin * 16 : nullptr};
  mark(0);
  // The index arrays are read before the wait for the preceding kernel (see DEC_PDL_TAIL): they are inputs
  // of the whole call chain, not something the kernel just before this one produces.
  const int ctx = __ldg(p.ctx_len + b);
  const int agent_raw = __ldg(p.agent_id + b);
  const bool use_lr = agent_raw >= 0;          // agent id -1: adapter-free view, base cache only
  const int agent = use_lr ? agent_raw : 0;
  __nv_bfloat16* out_bg = p.out + ((size_t)b * p.n_q + (size_t)g * G) * HD;
  // A context longer than the host's bound would index past the grid, the split and the block table:
  // rejected like a bad agent id (the same decision in every block of the request).
  if (ctx < 1 || ctx > p.max_ctx || agent_raw < -1 || agent_raw >= p.n_agents) {
    pdl_wait();               // `out` may still be read by the predecessor's consumers: store after the wait
    pdl_launch_dependents();
    if (split == 0) {
      if (raw_out) {
        // an empty shard (or a rejected request) contributes the neutral record: m = -big, l = 0, O' = 0
        float* rec = raw_out + ((size_t)b * p.n_kv + g) * C::PART_STRIDE;
        for (int i = threadIdx.x; i < C::PART_STRIDE; i += NT) rec[i] = i < 8 ? NEG_BIG : 0.f;
      } else {
        for (int i = threadIdx.x; i < G * HD; i += NT) out_bg[i] = __float2bfloat16(0.f);
      }
      if (threadIdx.x == 0 && ctx >= 1) atomicOr(p.status, StatusBits::BAD_INDEX);
    }
    return;
  }
  const int n_tiles = (ctx + PAGE - 1) / PAGE;
  const int n_splits = (n_tiles + p.chunk_tiles - 1) / p.chunk_tiles;
  if (split >= n_splits) return;
  const int tile0 = split * p.chunk_tiles;
  const int tile_end = min(n_tiles, tile0 + p.chunk_tiles);
  mark(1);
  if (ROPE && ctx > p.max_pos && threadIdx.x == 0) atomicOr(p.status, StatusBits::BAD_INDEX);   // positions are clamped
  decode_stream_block<HD, RK, RV, DEC_WARPS, ROPE>(p, smem, b, g, ctx, agent, use_lr, tile0, tile_end, mark);

  float* res = reinterpret_cast<float*>(smem);          // [m[8] | l[8] | O'[G][OW]]
  const int n_el = G * OW;
  const int rec_f = 16 + n_el;                          // used floats per record (multiple of 4)
  const int region = C::ticket_smem(p.stages) - 64;     // bytes of shared memory usable below
  const int bv_bytes = RV * HD * 2;
  unsigned char* bv_s = smem + region - bv_bytes;       // B_v[a][:, g] slice, [RV][HD] bf16
  const __nv_bfloat16* Bv = RV > 0 ? p.B_v + ((size_t)agent * RV) * ((size_t)p.n_kv * HD) + (size_t)g * HD : nullptr;
  auto stage_bv = [&]() {
    if constexpr (RV > 0) {
      for (int c = threadIdx.x; c < RV * (HD / 8); c += NT) {
        const int j = c / (HD / 8), ch = c % (HD / 8);
        cp_async16(smem_u32(bv_s) + c * 16, Bv + (size_t)j * p.n_kv * HD + ch * 8, 16);
      }
    }
  };
  float* fo = res + 16;                                 // final O' [G][OW]
  __shared__ float fin_l[8];
  __shared__ float fin_m[8];
  if (n_splits > 1) {
    float* rec = p.part + (((size_t)b * p.n_kv + g) * p.max_splits + split) * C::PART_STRIDE;
    for (int i = threadIdx.x; i < rec_f / 4; i += NT)
      reinterpret_cast<float4*>(rec)[i] = reinterpret_cast<const float4*>(res)[i];
    __syncthreads();
    __shared__ int is_last;
    if (threadIdx.x == 0) {
      // acq_rel at gpu scope: publishes this block's record (the barrier above orders the other
      // threads' stores before it) and, for the last arriver, acquires everybody else's
      int old;
      asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(p.tickets + (size_t)b * p.n_kv + g) : "memory");
      is_last = (old == n_splits - 1);
      if (is_last) p.tickets[(size_t)b * p.n_kv + g] = 0;   // ready for the next call
    }
    __syncthreads();
    mark(6);
    if (!is_last) return;
    // The last block merges all splits in split order, so the result does not depend on which
    // block that is.  Records (and the B_v slice) are staged with one batch of async copies, so the
    // L2 round trip is paid once.
    const float* base = p.part + (((size_t)b * p.n_kv + g) * p.max_splits) * C::PART_STRIDE;
    float* recs = res + 16 + 8 * OW;                    // [n_splits][rec_f] (staged) or [n_splits][16]
    const bool staged = (16 + 8 * OW + n_splits * rec_f + DEC_WARPS * n_el) * 4 + bv_bytes <= region;
    if (!raw_out) stage_bv();
    if (staged) {
      const int cpr = rec_f / 4;                        // 16-byte chunks per record
      for (int c = threadIdx.x; c < n_splits * cpr; c += NT) {
        const int s2 = c / cpr, ch = c % cpr;
        cp_async16(smem_u32(recs) + c * 16, base + (size_t)s2 * C::PART_STRIDE + ch * 4, 16);
      }
    } else {
      for (int i = threadIdx.x; i < n_splits * 16; i += NT)
        recs[i] = __ldcg(base + (size_t)(i >> 4) * C::PART_STRIDE + (i & 15));
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();
    mark(8);
    const int wstr = staged ? rec_f : 16;               // stride of the (m | l) heads kept in shared memory
    // weights: warp w owns query rows w, w+4 (< G); lanes stride over the splits
    for (int h = warp; h < G; h += DEC_WARPS) {
      float M = NEG_BIG;
      for (int s2 = lane; s2 < n_splits; s2 += 32) M = fmaxf(M, recs[s2 * wstr + h]);
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, d));
      float L = 0.f;
      for (int s2 = lane; s2 < n_splits; s2 += 32) {
        const float wv = fast_exp2(recs[s2 * wstr + h] - M);
        L += recs[s2 * wstr + 8 + h] * wv;
        recs[s2 * wstr + h] = wv;
      }
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) L += __shfl_xor_sync(0xffffffffu, L, d);   // fixed tree: deterministic
      if (lane == 0) { fin_l[h] = L; fin_m[h] = M; }
    }
    __syncthreads();
    mark(9);
    // merge: a thread owns one float4 column of O' and a quarter of the splits (s = q, q+4, ...),
    // four loads in flight; the quarters are then added in a fixed order
    const int n_f4 = n_el / 4;
    float* wsum = recs + (size_t)n_splits * wstr;       // [4][n_el]
    for (int item = threadIdx.x; item < 4 * n_f4; item += NT) {
      const int col = item % n_f4, qd = item / n_f4;
      const int h = (col * 4) / OW;
      float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
      auto fetch = [&](int s2) -> float4 {
        if (staged) return *reinterpret_cast<const float4*>(recs + (size_t)s2 * rec_f + 16 + col * 4);
        return __ldcg(reinterpret_cast<const float4*>(base + (size_t)s2 * C::PART_STRIDE + 16 + col * 4));
      };
      int s2 = qd;
      for (; s2 + 4 < n_splits; s2 += 8) {
        const float4 x0 = fetch(s2), x1 = fetch(s2 + 4);
        const float w0 = recs[s2 * wstr + h], w1 = recs[(s2 + 4) * wstr + h];
        a0.x += x0.x * w0; a0.y += x0.y * w0; a0.z += x0.z * w0; a0.w += x0.w * w0;
        a1.x += x1.x * w1; a1.y += x1.y * w1; a1.z += x1.z * w1; a1.w += x1.w * w1;
      }
      if (s2 < n_splits) {
        const float4 x0 = fetch(s2);
        const float w0 = recs[s2 * wstr + h];
        a0.x += x0.x * w0; a0.y += x0.y * w0; a0.z += x0.z * w0; a0.w += x0.w * w0;
      }
      *reinterpret_cast<float4*>(wsum + (size_t)qd * n_el + col * 4) =
          make_float4(a0.x + a1.x, a0.y + a1.y, a0.z + a1.z, a0.w + a1.w);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n_el; e += NT)
      fo[e] = ((wsum[e] + wsum[n_el + e]) + wsum[2 * n_el + e]) + wsum[3 * n_el + e];
  } else {
    if (!raw_out) stage_bv();
    cp_async_commit();
    if (threadIdx.x < 8) { fin_l[threadIdx.x] = res[8 + threadIdx.x]; fin_m[threadIdx.x] = res[threadIdx.x]; }
    cp_async_wait<0>();
  }
  __syncthreads();
  mark(10);
  if (raw_out) {
    // partial-output mode: the merged record of this (request, kv head) over the LOCAL tokens, not
    // normalised and without the value-side epilogue; a later combine step merges such records
    float* rec = raw_out + ((size_t)b * p.n_kv + g) * C::PART_STRIDE;
    for (int i = threadIdx.x; i < C::PART_STRIDE; i += NT) {
      float v = 0.f;
      if (i < 8) v = i < G ? fin_m[i] : NEG_BIG;
      else if (i < 16) v = i - 8 < G ? fin_l[i - 8] : 0.f;
      else if (i - 16 < n_el) v = fo[i - 16];
      rec[i] = v;
    }
    mark(7);
    return;
  }
  const __nv_bfloat16* bvs = reinterpret_cast<const __nv_bfloat16*>(bv_s);
  for (int e = threadIdx.x; e < G * HD; e += NT) {
    const int h = e / HD, c = e % HD;
    float v = fo[h * OW + c];
    if constexpr (RV > 0) {
      float u = 0.f;
#pragma unroll 8
      for (int j = 0; j < RV; ++j) u += fo[h * OW + HD + j] * __bfloat162float(bvs[j * HD + c]);
      v += p.s_v * u;
    }
    out_bg[e] = __float2bfloat16(v / fin_l[h]);
  }
  mark(7);
}

// ------------------------------------------------------------------------------------------------
// Cluster kernel: grid (cluster size CS, kv head, request), cluster (CS,1,1), NW warps.
//
// Merge.  Block `o` finishes the output columns [o cols, o cols + ncol) of the (b, g) unit.  Every block
// merges the records of its own warps, adds the value-side adapter term to its partial (the term is linear in
// the partial: s_v U B_v of the merged sum equals the sum of the per-block terms), and SENDS each merged value
// to the block that owns its column with st.async, which also counts the bytes on an mbarrier in the owner's
// shared memory; (m, l) of every head go to every owner.  An owner waits for its byte count, then weighs and
// adds the CS contributions in rank order and stores.  The only cluster-wide barrier is the one that makes the
// mbarriers' initialisation visible: arrived at when the kernel starts, waited for before the first send, i.e.
// long complete.  A block leaves once it has received everything addressed to it, so no send can reach the
// shared memory of a block that is gone.
// MINB = 2 (8 warps, head_dim 64): 16-block clusters need two blocks per SM, which caps the kernel at 128
// registers; the one-block-per-SM ring layout uses the MINB = 1 instance, free of that cap.
template <int HD, int RK, int RV, int NW, bool ROPE = false, int MINB = 1>
__global__ void __launch_bounds__(NW * 32, MINB)
lr_attend_decode_cluster_kernel(const DecodeParams p) {
  using C = DecodeCfg<HD, RK, RV>;
  float* const raw_out = ROPE ? nullptr : p.raw;      // no rotary partial-output entry point: compiled out there
  constexpr int OW = C::OW;
  constexpr int OWP = C::OWP;
  constexpr int WREC = C::WREC;
  constexpr int NT = NW * 32;
  extern __shared__ __align__(128) unsigned char smem[];
  const int rank = blockIdx.x, CS = gridDim.x;          // the cluster spans grid.x
  const int g = blockIdx.y, b = blockIdx.z;
  const int G = p.group;
  const int cta_lin = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
  const DecodeTrace mark{p.trace ? p.trace + (size_t)cta_lin * 16 : nullptr};
  mark(0);
  mark.where();
  const int ctx = __ldg(p.ctx_len + b);        // index arrays: read before the wait for the preceding kernel
  const int agent_raw = __ldg(p.agent_id + b);
  const bool use_lr = agent_raw >= 0;          // agent id -1: adapter-free view, base cache only
  const int agent = use_lr ? agent_raw : 0;
  __nv_bfloat16* out_bg = p.out + ((size_t)b * p.n_q + (size_t)g * G) * HD;
  if (ctx < 1 || ctx > p.max_ctx || agent_raw < -1 || agent_raw >= p.n_agents) {   // the same decision in every block of the cluster
    pdl_wait();
    pdl_launch_dependents();
    if (rank == 0) {
      if (raw_out) {
        float* rec = raw_out + ((size_t)b * p.n_kv + g) * C::PART_STRIDE;   // neutral record: m = -big, l = 0, O' = 0
        for (int i = threadIdx.x; i < C::PART_STRIDE; i += NT) rec[i] = i < 8 ? NEG_BIG : 0.f;
      } else {
        for (int i = threadIdx.x; i < G * HD; i += NT) out_bg[i] = __float2bfloat16(0.f);
      }
      if (threadIdx.x == 0 && ctx >= 1) atomicOr(p.status, StatusBits::BAD_INDEX);
    }
    return;
  }
  const int n_tiles = (ctx + PAGE - 1) / PAGE;
  const int tile0 = min(n_tiles, rank * p.chunk_tiles);
  const int tile_end = min(n_tiles, tile0 + p.chunk_tiles);
  mark(1);
  // Columns of the merged record that are divided over the blocks: the head dimension (the LR-V coordinates are
  // spent inside each block), or the whole record in partial-output mode (no B_v there).
  const int W = raw_out ? OW : HD;
  const int cols = (W + CS - 1) / CS;                   // the cluster size need not divide W:
  const int c0 = rank * cols;
  const int ncol = max(0, min(cols, W - c0));           // the last blocks own fewer (or no) columns
  float* recv = reinterpret_cast<float*>(smem + C::cluster_core(NW, p.stages));
  const uint32_t recv_u32 = smem_u32(recv);
  const uint32_t recv_bar = recv_u32 + C::RECV_FLOATS * 4;
  const int ml_off = (CS * G * cols + 1) & ~1;          // floats; the (m, l) pairs are stored as 8-byte words
  const uint32_t bv_bar = recv_bar + 8;
  if (threadIdx.x == 0) {
    mbar_init(recv_bar, 1);
    if constexpr (C::WEXP) mbar_init(bv_bar, NT);         // every thread arrives once its copies of the B_v slice have landed
    if (ncol > 0) mbar_expect_tx(recv_bar, (uint32_t)(CS * G * (ncol + 2) * 4));   // the one arrival, and the bytes to come
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if constexpr (C::WEXP) __syncthreads(); else __syncwarp();   // bv_bar is used by this block's own threads right below
  cluster_arrive_relaxed();            // the fence above orders the initialisation; nothing else is published here
  // division by the run-time slice width, as a multiplication (exact for numerators below 1024)
  const uint32_t inv_cols = (65536u + (uint32_t)cols - 1u) / (uint32_t)cols;
  const bool expand = RV > 0 && use_lr && !raw_out && p.B_v != nullptr;
  // B_v[a][:, g] slice, requested now (before the page stream).  WEXP: copied to shared memory in the layout of a
  // value page (rows = rank coordinates, padded with zero rows to 16); each thread's arrival on bv_bar fires when
  // its copies have landed.  Otherwise: parked in registers, a unit being eight consecutive rank rows of one column
  // (one 16-byte word of the layout [RV / 8][HD][8] that the adapter term reads below).
  const uint32_t bv_u32 = smem_u32(smem + C::cluster_bv(NW, p.stages));
  constexpr int BVU = (RV > 0 && !C::WEXP) ? ((RV / 8) * HD + NT - 1) / NT : 1;
  uint4 bv_pre[BVU];
  if constexpr (RV > 0 && C::WEXP) {
    if (expand) {
      constexpr int CPR = HD / 8;
      const __nv_bfloat16* Bv = p.B_v + ((size_t)agent * RV) * ((size_t)p.n_kv * HD) + (size_t)g * HD;
      for (int i = threadIdx.x; i < C::BVP * CPR; i += NT) {
        const int j = i / CPR, ch = i % CPR;
        cp_async16(bv_u32 + swz_off<CPR>(j, ch), Bv + (size_t)(j < RV ? j : 0) * p.n_kv * HD + ch * 8, j < RV ? 16 : 0);
      }
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bv_bar) : "memory");
    }
  } else if constexpr (RV > 0) {
    const unsigned short* Bv = reinterpret_cast<const unsigned short*>(p.B_v + ((size_t)agent * RV) * ((size_t)p.n_kv * HD) + (size_t)g * HD);
    const size_t rs = (size_t)p.n_kv * HD;
#pragma unroll
    for (int k = 0; k < BVU; ++k) {
      const int i = threadIdx.x + k * NT;                 // unit (q, c) = (i / HD, i % HD): rows 8q .. 8q+7 of column c
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (expand && i < (RV / 8) * HD) {
        const unsigned short* src = Bv + (size_t)(i / HD) * 8 * rs + (i % HD);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          w[j] = (uint32_t)__ldg(src + (2 * j) * rs) | ((uint32_t)__ldg(src + (2 * j + 1) * rs) << 16);
      }
      bv_pre[k] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
  if (ROPE && ctx > p.max_pos && threadIdx.x == 0) atomicOr(p.status, StatusBits::BAD_INDEX);   // positions are clamped
  decode_stream_block<HD, RK, RV, NW, ROPE, false>(p, smem, b, g, ctx, agent, use_lr, tile0, tile_end, mark,
                                                   WarpExpand{C::WEXP && expand, bv_u32, bv_bar});

  // ---- the warps' records are at the start of shared memory.  WEXP: their first hd columns are final (the adapter
  //      term is in), the LR-V columns matter in partial-output mode only.  Otherwise the B_v slice and the merged
  //      LR-V coordinates are placed behind the records and the term is added after the block merge.
  constexpr bool TAIL_EXPAND = RV > 0 && !C::WEXP;
  const int Wm = (TAIL_EXPAND || raw_out) ? OW : HD;    // merged columns per head
  float* mg = reinterpret_cast<float*>(smem);
  uint4* bvs = reinterpret_cast<uint4*>(smem + C::merge_bytes(NW));                  // [RV / 8][HD] words of 8 bf16 (rank rows 8q .. 8q+7)
  float* lrm = reinterpret_cast<float*>(smem + C::merge_bytes(NW) + RV * HD * 2);   // [8][RV]
  if constexpr (TAIL_EXPAND) {
    if (expand) {
#pragma unroll
      for (int k = 0; k < BVU; ++k) {
        const int i = threadIdx.x + k * NT;
        if (i < (RV / 8) * HD) bvs[i] = bv_pre[k];
      }
    }
  }
  __syncthreads();
  mark(13);
  // every thread merges its own elements and derives the warp weights of its query row itself; element
  // G*Wm + h is the pair (m, l) of row h
  const int n_el = G * Wm;
  auto head_col = [&](int e, int& h, int& c) {           // constant divisors
    if (Wm == HD) { h = e / HD; c = e % HD; } else { h = e / OW; c = e % OW; }
  };
  // The thread of element (h, c) with c < CS also merges the denominator of row h - its weights are at hand - and
  // will send the pair (m, l) to block c (head_dim >= 64 > CS: such a thread exists for every receiving block).
  constexpr int PER_THREAD = (8 * OW + NT - 1) / NT;
  float acc[PER_THREAD], acc_m[PER_THREAD], acc_l[PER_THREAD];
#pragma unroll
  for (int k = 0; k < PER_THREAD; ++k) {
    const int e = threadIdx.x + k * NT;
    float v = 0.f, M = NEG_BIG, L = 0.f;
    if (e < n_el) {
      int h, c;
      head_col(e, h, c);
      const int src = 16 + h * OWP + c;
      float mw[NW], xw[NW];
#pragma unroll
      for (int w = 0; w < NW; ++w) { mw[w] = mg[w * WREC + h]; xw[w] = mg[w * WREC + src]; }
#pragma unroll
      for (int w = 0; w < NW; ++w) M = fmaxf(M, mw[w]);
#pragma unroll
      for (int w = 0; w < NW; ++w) mw[w] = fast_exp2(mw[w] - M);
#pragma unroll
      for (int w = 0; w < NW; ++w) v += xw[w] * mw[w];                  // warp order: deterministic
      if (c < CS) {
#pragma unroll
        for (int w = 0; w < NW; ++w) L += mg[w * WREC + 8 + h] * mw[w];
      }
      if constexpr (TAIL_EXPAND) {
        if (expand && c >= HD) lrm[h * RV + c - HD] = v;
      }
    }
    acc[k] = v; acc_m[k] = M; acc_l[k] = L;
  }
  if constexpr (TAIL_EXPAND) {
    if (expand) __syncthreads();       // block-uniform: the merged LR-V coordinates are complete
  }
  mark(14);
#pragma unroll
  for (int k = 0; k < PER_THREAD; ++k) {
    const int e = threadIdx.x + k * NT;
    if (e < n_el) {
      int h, c;
      head_col(e, h, c);
      if (c < CS && c * cols < W)                    // every block that owns columns needs every block's (m, l)
        st_async_f32x2(dsmem_addr(recv_u32 + (uint32_t)((ml_off + (rank * G + h) * 2) * 4), c), acc_m[k], acc_l[k],
                       dsmem_addr(recv_bar, c));
      if (c < W) {
        float v = acc[k];
        if constexpr (TAIL_EXPAND) {
          if (expand) {                // value-side adapter term of this block's partial: s_v sum_j U[h][j] B_v[j][c]
            float u[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int q = 0; q < RV / 8; ++q) {
              const uint4 bw = bvs[q * HD + c];
              const float4 ua = *reinterpret_cast<const float4*>(lrm + h * RV + q * 8);
              const float4 ub = *reinterpret_cast<const float4*>(lrm + h * RV + q * 8 + 4);
              u[0] += ua.x * __uint_as_float(bw.x << 16);
              u[1] += ua.y * __uint_as_float(bw.x & 0xffff0000u);
              u[2] += ua.z * __uint_as_float(bw.y << 16);
              u[3] += ua.w * __uint_as_float(bw.y & 0xffff0000u);
              u[0] += ub.x * __uint_as_float(bw.z << 16);
              u[1] += ub.y * __uint_as_float(bw.z & 0xffff0000u);
              u[2] += ub.z * __uint_as_float(bw.w << 16);
              u[3] += ub.w * __uint_as_float(bw.w & 0xffff0000u);
            }
            v += p.s_v * ((u[0] + u[1]) + (u[2] + u[3]));
          }
        }
        const int owner = (int)(((uint32_t)c * inv_cols) >> 16);
        st_async_f32(dsmem_addr(recv_u32 + (uint32_t)(((rank * G + h) * cols + (c - owner * cols)) * 4), owner), v,
                     dsmem_addr(recv_bar, owner));
      }
    }
  }
  mark(6);
  if (ncol == 0) { mark(7); return; }  // nothing is addressed to a block without columns
  // Four lanes share an element (h, c) of this block's slice, lane `sub` taking the sources sub, sub + 4, sub + 8,
  // sub + 12; the indices are worked out before the wait, so that loads, a short chain and two shuffle rounds are
  // all that follows it.  The order of every sum is fixed: results do not depend on timing.
  const float* ml = recv + ml_off;
  const int sub = threadIdx.x & 3;
  const int n_own = G * ncol;
  int el = threadIdx.x >> 2;
  int h = el / ncol, c = el - h * ncol;
  mbar_wait_cluster(recv_bar, 0, p.status);
  mark(12);
  float* rec = raw_out ? raw_out + ((size_t)b * p.n_kv + g) * C::PART_STRIDE : nullptr;
  for (int base = 0; base < n_own; base += NT / 4) {
    const bool live = el < n_own;
    const int hh = live ? h : 0, cc = live ? c : 0;
    float mr[4], lr[4], xr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = sub + 4 * i;
      if (r < CS) {
        const float2 t = *reinterpret_cast<const float2*>(ml + (r * G + hh) * 2);
        mr[i] = t.x; lr[i] = t.y; xr[i] = recv[(r * G + hh) * cols + cc];
      } else {
        mr[i] = NEG_BIG; lr[i] = 0.f; xr[i] = 0.f;
      }
    }
    float M = fmaxf(fmaxf(mr[0], mr[1]), fmaxf(mr[2], mr[3]));
    M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 1));
    M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 2));
    float v = 0.f, L = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float w = fast_exp2(mr[i] - M); v += xr[i] * w; L += lr[i] * w; }
    v += __shfl_xor_sync(0xffffffffu, v, 1); L += __shfl_xor_sync(0xffffffffu, L, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2); L += __shfl_xor_sync(0xffffffffu, L, 2);
    if (live && sub == 0) {
      if (rec) rec[16 + hh * OW + c0 + cc] = v;          // partial-output mode: merged, un-normalised
      else out_bg[hh * HD + c0 + cc] = __float2bfloat16(v / L);
    }
    el += NT / 4;
    if (base + NT / 4 < n_own) { h = el / ncol; c = el - h * ncol; }   // only if another pass follows
  }
  if (rec && rank == 0) {                               // block 0 adds the maxima, the denominators and the unused slots
    for (int e = G * OW + threadIdx.x; e < 8 * OW; e += NT) rec[16 + e] = 0.f;
    if (threadIdx.x < 8) {
      float M = NEG_BIG, L = 0.f;
      if (threadIdx.x < G) {
        for (int r = 0; r < CS; ++r) M = fmaxf(M, ml[(r * G + threadIdx.x) * 2]);
        // the same tree as above: sources r, r + 4, r + 8, r + 12 first, then pairs of those partial sums
        float part[4] = {0.f, 0.f, 0.f, 0.f};
        for (int r = 0; r < CS; ++r) part[r & 3] += ml[(r * G + threadIdx.x) * 2 + 1] * fast_exp2(ml[(r * G + threadIdx.x) * 2] - M);
        L = (part[0] + part[1]) + (part[2] + part[3]);
      }
      rec[threadIdx.x] = M;
      rec[8 + threadIdx.x] = L;
    }
  }
  mark(7);
}

}  // namespace precc
