// Skinny projection GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
//   C[M, N_out] = X[M, K] . Wt[N_out, K]^T        (both operands K-major bf16, fp32 accumulate)
//
// with a scatter epilogue that writes bf16 rows straight into the paged caches:
//   mode 0  LR precompute (Section 3.1):  column -> (projection, agent, r index), LR cache rows
//   mode 1  base projection (Section 3.2): column -> (projection, kv head, c), base cache rows
//   mode 2  both at once: the first 2*n_kv*hd columns go to the base caches, the rest to the LR caches
//           (the hidden states of a newly processed segment are read once, Section 3.1)
//
// Persistent blocks, 128 x BN output tiles.  Warp roles: warp 0 = TMA producer (one lane), warp 1 =
// TMEM owner + MMA issuer (one lane), warps 2..5 = epilogue (one TMEM lane = one row each).  A
// STAGES-deep ring of {X tile 128x64, Wt tile BNx64} in 128-byte-swizzled shared memory is handed from
// producer to issuer with mbarriers; tcgen05.commit releases a stage when its MMAs have read it.  The
// accumulator is double-buffered in TMEM (2 x BN columns), so a tile's epilogue overlaps the next
// tile's MMAs.
// Every wait is bounded: on expiry the waiter records PRECC_STATUS_TIMEOUT and carries on, so the
// kernel always terminates and frees its TMEM.
#pragma once
#include "tc_common.cuh"

namespace precc {

// Routes eight consecutive output columns [gc, gc+8) of one row (cache block `blk`, offset `off`) to
// their place in the paged caches: column -> (projection, head, c) for base columns, (projection, agent,
// r) for LR columns (skipped when the agent's bit in `mask` — the call's mask or the row's own — is clear).  Pieces never straddle a destination row
// because head_dim and the ranks are multiples of 8.
// `gm` is the row's index in the call (for the optional second LR destination of that row, see lr_copy_slots).
__device__ __forceinline__ void store_piece(const GemmParams& p, long long blk, int off, int gc, const float (&v8)[8],
                                            unsigned long long mask, int gm) {
  const int w = p.n_kv * p.hd;
  __nv_bfloat16* dst;
  __nv_bfloat16* dst2 = nullptr;
  const bool to_base = p.mode == 1 || (p.mode == 2 && gc < 2 * w);
  if (!to_base) {
    const int n_k = p.n_agents * p.rank_k;
    const int gl = p.mode == 2 ? gc - 2 * w : gc;
    const bool is_v = gl >= n_k;
    const int rr = is_v ? p.rank_v : p.rank_k;
    const int cc = is_v ? gl - n_k : gl;
    const int sh = is_v ? p.rv_shift : p.rk_shift;
    const int agent = cc >> sh, ri = cc & (rr - 1);
    if (!((mask >> agent) & 1ull)) return;
    dst = (is_v ? p.lr_v : p.lr_k) + (((long long)agent * p.n_blocks + blk) * PAGE + off) * rr + ri;
    if (p.lr_copy_slots) {
      const long long s2 = p.lr_copy_slots[gm];
      if (s2 >= p.n_blocks * PAGE) atomicOr(p.status, StatusBits::BAD_INDEX);
      else if (s2 >= 0) dst2 = (is_v ? p.lr_v : p.lr_k) + ((long long)agent * p.n_blocks * PAGE + s2) * rr + ri;
    }
  } else {
    const bool is_v = gc >= w;
    const int cc = is_v ? gc - w : gc;
    const int g = cc >> p.hd_shift, c = cc & (p.hd - 1);
    dst = (is_v ? p.base_v : p.base_k) + ((blk * p.n_kv + g) * PAGE + off) * p.hd + c;
  }
  uint4 v;
  v.x = pack_bf16(v8[0], v8[1]);
  v.y = pack_bf16(v8[2], v8[3]);
  v.z = pack_bf16(v8[4], v8[5]);
  v.w = pack_bf16(v8[6], v8[7]);
  *reinterpret_cast<uint4*>(dst) = v;
  if (dst2) *reinterpret_cast<uint4*>(dst2) = v;
}

// Epilogue of one output tile for one warp: TMEM lane = tile row (this warp owns lanes lane_base .. lane_base + 31 of
// the accumulator at `tmem_tile`, which holds rows m0 .. m0 + 127 and columns n0 .. n0 + BN - 1).  Waits for the
// accumulator (bounded), converts to bf16 and routes 16-byte pieces to the paged caches; key columns of the rotary
// variant are rotated by the row's position first.
// The epilogue shares its SM's issue slots with the lanes that feed the tensor pipe, so it is kept lean: what depends
// on the row (its slot -> element offsets into the base and LR arrays, its agent mask, its optional second LR
// destination) is computed once per tile, what depends on the column (projection, head or agent, offset inside the
// destination row) is the same for every lane and uses shifts (head_dim and the ranks are powers of two).
__device__ __forceinline__ void gemm_epilogue_tile(const GemmParams& p, uint32_t tmem_tile, int m0, int n0, int lane_base, int lane,
                                                   uint32_t acc_full_bar, uint32_t parity) {
  const int row = lane_base + lane;
  const int hs = p.hd_shift;
  const int w = p.n_kv << hs;
  const int gm = m0 + row;
  bool row_ok = gm < p.M;
  long long slot = 0;
  if (row_ok) {
    slot = p.slot_mapping ? (long long)p.slot_mapping[gm] : p.start_slot + gm;
    if (slot < 0 || slot >= p.n_blocks * PAGE) { atomicOr(p.status, StatusBits::BAD_INDEX); row_ok = false; slot = 0; }
  }
  const long long blk = slot / PAGE;
  const int off = (int)(slot % PAGE);
  const unsigned long long row_mask = (p.row_masks && row_ok) ? p.row_masks[gm] : p.agent_mask;
  long long slot2 = -1;                               // second destination of this row's LR pieces, if any
  if (p.lr_copy_slots && row_ok) {
    slot2 = p.lr_copy_slots[gm];
    if (slot2 >= p.n_blocks * PAGE) { atomicOr(p.status, StatusBits::BAD_INDEX); slot2 = -1; }
  }
  long long pos = 0;
  if (p.rope && row_ok) {
    pos = p.positions ? (long long)p.positions[gm] : p.start_pos + gm;
    if (pos < 0 || pos >= p.max_pos) { atomicOr(p.status, StatusBits::BAD_INDEX); row_ok = false; }
  }
  // element offsets of this row inside the base arrays ([blk][g][off][c]: the head term is added per column) and
  // inside one agent's LR arrays ([blk][off][r] = [slot][r])
  const long long base_row = ((blk * p.n_kv * PAGE) + off) << hs;
  const int n_k = p.n_agents << p.rk_shift;           // LR-K columns of the call (0 when rank_k == 0: n_agents << 0 is not used then)
  const int n_lrk = p.rank_k > 0 ? n_k : 0;
  mbar_wait_relaxed(acc_full_bar, parity, p.status);
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  for (int c0 = 0; c0 < p.BN && n0 + c0 < p.N_out; c0 += 16) {
    if (p.rope && n0 + c0 < w) {
      // key columns: chunk [c, c+16) of the lower half of a head together with its partner chunk
      const int gc = n0 + c0;
      const int g = gc >> hs, c = gc & (p.hd - 1);
      if (c >= p.hd / 2) continue;                  // done with its partner
      uint32_t lo[16], hi[16];
      tmem_ld16(tmem_tile + (static_cast<uint32_t>(lane_base) << 16) + c0, lo);
      tmem_ld16(tmem_tile + (static_cast<uint32_t>(lane_base) << 16) + c0 + p.hd / 2, hi);
      asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
      if (!row_ok) continue;
      const float4* cs = p.rope + pos * (p.hd / 4) + c / 2;
      uint32_t ol[8], oh[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const float4 t4 = __ldg(cs + k);
        const float l0 = __uint_as_float(lo[2 * k]), l1 = __uint_as_float(lo[2 * k + 1]);
        const float h0 = __uint_as_float(hi[2 * k]), h1 = __uint_as_float(hi[2 * k + 1]);
        ol[k] = pack_bf16(l0 * t4.x - h0 * t4.y, l1 * t4.z - h1 * t4.w);
        oh[k] = pack_bf16(h0 * t4.x + l0 * t4.y, h1 * t4.z + l1 * t4.w);
      }
      __nv_bfloat16* dst = p.base_k + base_row + ((long long)(g * PAGE) << hs) + c;
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(ol[0], ol[1], ol[2], ol[3]);
      reinterpret_cast<uint4*>(dst)[1] = make_uint4(ol[4], ol[5], ol[6], ol[7]);
      reinterpret_cast<uint4*>(dst + p.hd / 2)[0] = make_uint4(oh[0], oh[1], oh[2], oh[3]);
      reinterpret_cast<uint4*>(dst + p.hd / 2)[1] = make_uint4(oh[4], oh[5], oh[6], oh[7]);
      continue;
    }
    uint32_t r[16];
    tmem_ld16(tmem_tile + (static_cast<uint32_t>(lane_base) << 16) + c0, r);
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
    if (!row_ok) continue;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int gc = n0 + c0 + 8 * h;               // the same for every lane: the routing below is warp-uniform
      if (gc >= p.N_out) break;
      uint4 v;
      v.x = pack_bf16(__uint_as_float(r[8 * h + 0]), __uint_as_float(r[8 * h + 1]));
      v.y = pack_bf16(__uint_as_float(r[8 * h + 2]), __uint_as_float(r[8 * h + 3]));
      v.z = pack_bf16(__uint_as_float(r[8 * h + 4]), __uint_as_float(r[8 * h + 5]));
      v.w = pack_bf16(__uint_as_float(r[8 * h + 6]), __uint_as_float(r[8 * h + 7]));
      if (p.mode == 1 || (p.mode == 2 && gc < 2 * w)) {
        const bool is_v = gc >= w;
        const int cc = is_v ? gc - w : gc;
        const int g = cc >> hs, c = cc & (p.hd - 1);
        __nv_bfloat16* dst = (is_v ? p.base_v : p.base_k) + base_row + ((long long)(g * PAGE) << hs) + c;
        *reinterpret_cast<uint4*>(dst) = v;
      } else {
        const int gl = p.mode == 2 ? gc - 2 * w : gc;
        const bool is_v = gl >= n_lrk;
        const int sh = is_v ? p.rv_shift : p.rk_shift;
        const int cc = is_v ? gl - n_lrk : gl;
        const int agent = cc >> sh, ri = cc & ((1 << sh) - 1);
        if (!((row_mask >> agent) & 1ull)) continue;
        __nv_bfloat16* arr = (is_v ? p.lr_v : p.lr_k) + (((long long)agent * p.n_blocks * PAGE) << sh) + ri;
        *reinterpret_cast<uint4*>(arr + (slot << sh)) = v;
        if (slot2 >= 0) *reinterpret_cast<uint4*>(arr + (slot2 << sh)) = v;
      }
    }
  }
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
proj_gemm_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the 128-byte swizzle atoms
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int b_bytes = p.BN * GEMM_BK * 2;
  const int stage_bytes = GEMM_A_BYTES + b_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes);
  // barrier map: full[stages] | empty[stages] | acc_full[2] | acc_empty[2]
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = full0 + 8 * p.stages;
  const uint32_t acc_full = empty0 + 8 * p.stages;
  const uint32_t acc_empty = acc_full + 16;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb = p.K / GEMM_BK;
  const int n_tiles_n = (p.N_out + p.BN - 1) / p.BN;
  // Row tiles.  With a single column tile the kernel is HBM-bound on X, and a row-tile count that is not a
  // multiple of the grid leaves part of the machine idle in the last round (256 tiles on 148 blocks = 1.73
  // rounds).  Then the count is rounded up to a multiple of the grid and the tiles are spread evenly over
  // the rows: neighbours overlap by a few rows, which are computed twice with identical results (the
  // overlap is re-read from L2, not from DRAM), and every block streams the same number of rows.
  const int m_plain = (p.M + GEMM_BM - 1) / GEMM_BM;
  const bool spread = p.spread_rows && n_tiles_n == 1 && m_plain > (int)gridDim.x && p.M >= GEMM_BM;
  const int m_tiles = spread ? ((m_plain + (int)gridDim.x - 1) / (int)gridDim.x) * (int)gridDim.x : m_plain;
  const int n_tiles = m_tiles * n_tiles_n;
  auto row0_of = [&](int mt) -> int {
    if (!spread) return mt * GEMM_BM;
    return (int)(((long long)mt * (p.M - GEMM_BM)) / (m_tiles - 1));   // first tile at 0, last one ends at M
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(acc_full, 1); mbar_init(acc_full + 8, 1);
    mbar_init(acc_empty, 4); mbar_init(acc_empty + 8, 4);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_holder)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  // Persistent: this block takes tiles blockIdx.x, blockIdx.x + gridDim.x, ...; the column tile index
  // runs fastest, so blocks working at the same time share their row tile of X in L2.  The shared
  // memory ring runs straight through tile boundaries and the accumulator is double-buffered in TMEM,
  // so the epilogue of one tile overlaps the MMAs of the next.
  if (warp == 0) {
    if (lane == 0) {
      int it = 0;
      for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int m0 = row0_of(t / n_tiles_n), n0 = (t % n_tiles_n) * p.BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % p.stages;
          if (it >= p.stages) mbar_wait(empty0 + 8 * s, ((it / p.stages) - 1) & 1, p.status);
          GEMM_STAMP(p, it, 0);
          const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
          mbar_expect_tx(full0 + 8 * s, stage_bytes);
          tma_load_2d(sa, &map_x, kb * GEMM_BK, m0, full0 + 8 * s);
          tma_load_3d(sa + GEMM_A_BYTES, &map_w, 0, n0, kb, full0 + 8 * s);      // packed weights are k-blocked
          GEMM_STAMP(p, it, 1);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(p.BN);
      const uint64_t da0 = umma_desc_sw128(smem_u32(smem));
      const uint64_t db0 = umma_desc_sw128(smem_u32(smem) + GEMM_A_BYTES);
      int it = 0, i = 0;
      for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++i) {
        const int buf = i & 1;
        if (i >= 2) mbar_wait(acc_empty + 8 * buf, ((i >> 1) - 1) & 1, p.status);   // epilogue has drained this buffer
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint32_t d = tmem_base + buf * p.BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % p.stages;
          mbar_wait(full0 + 8 * s, (it / p.stages) & 1, p.status);
          GEMM_STAMP(p, it, 2);
          asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
          const uint64_t so = (uint64_t)((s * stage_bytes) >> 4);
#pragma unroll
          for (int k = 0; k < GEMM_BK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per step
            umma_bf16(d, da0 + so + 2 * k, db0 + so + 2 * k, idesc, (kb | k) ? 1u : 0u);
          GEMM_STAMP(p, it, 3);
          umma_commit(empty0 + 8 * s);             // stage reusable once these MMAs have read it
          GEMM_STAMP(p, it, 4);
        }
        umma_commit(acc_full + 8 * buf);           // accumulator of this tile complete
      }
    }
  } else {
    // ---- epilogue: TMEM lane = tile row; this warp may touch lanes 32*(warp%4) .. +31
    const int lane_base = (warp & 3) * 32;
    int i = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++i) {
      const int buf = i & 1;
      const int m0 = row0_of(t / n_tiles_n), n0 = (t % n_tiles_n) * p.BN;
      gemm_epilogue_tile(p, tmem_base + buf * p.BN, m0, n0, lane_base, lane, acc_full + 8 * buf, (i >> 1) & 1);
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(acc_empty + 8 * buf) : "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}


// Reduce step of the split-K kernel: thread t of the block's 192 threads takes the 16-byte pieces t, t + 192, ...
// of this block's slice (piece f = row * cw/4 + q), 16 / KS of them at a time, so that sixteen loads over
// distributed shared memory are in flight per thread; consecutive lanes read consecutive pieces of a peer; the
// peers are summed in rank order.  The odd piece of a pair hands its four columns to the even one, which
// stores eight.
template <int KS>
__device__ __forceinline__ void splitk_reduce(const GemmParams& p, uint32_t smem_base, int rank, int cw, int m0, int n0, int t) {
  constexpr int G = 16 / KS;
  const int XS = cw + 4, qpr = cw / 4;
  const uint32_t slice = smem_base + (uint32_t)rank * GEMM_BM * XS * 4;
  const int total = GEMM_BM * qpr;                              // a multiple of 128
  for (int f0 = t; f0 < total; f0 += GEMM_THREADS * G) {
    float4 a[G][KS];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const int f = f0 + g * GEMM_THREADS;
      const int row = f / qpr, q = f % qpr;
#pragma unroll
      for (int r = 0; r < KS; ++r) {
        if (f < total && m0 + row < p.M) {                        // rows past M are never stored: not fetched either
          uint32_t remote;
          asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote) : "r"(slice + (uint32_t)(row * XS + 4 * q) * 4), "r"(r));
          asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];\n" : "=f"(a[g][r].x), "=f"(a[g][r].y), "=f"(a[g][r].z), "=f"(a[g][r].w) : "r"(remote));
        } else {
          a[g][r] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const int f = f0 + g * GEMM_THREADS;
      const int row = f / qpr, q = f % qpr;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int r = 0; r < KS; ++r) { v.x += a[g][r].x; v.y += a[g][r].y; v.z += a[g][r].z; v.w += a[g][r].w; }
      const float4 hi = make_float4(__shfl_down_sync(0xffffffffu, v.x, 1), __shfl_down_sync(0xffffffffu, v.y, 1),
                                    __shfl_down_sync(0xffffffffu, v.z, 1), __shfl_down_sync(0xffffffffu, v.w, 1));
      if ((q & 1) == 0 && f < total) {
        const int gm = m0 + row, c = rank * cw + 4 * q, gc = n0 + c;
        if (gm < p.M && c < p.BN && gc < p.N_out) {
          const long long slot = p.slot_mapping ? (long long)p.slot_mapping[gm] : p.start_slot + gm;
          if (slot < 0 || slot >= p.n_blocks * PAGE) {
            atomicOr(p.status, StatusBits::BAD_INDEX);
          } else {
            const float v8[8] = {v.x, v.y, v.z, v.w, hi.x, hi.y, hi.z, hi.w};
            store_piece(p, slot / PAGE, (int)(slot % PAGE), gc, v8, p.row_masks ? p.row_masks[gm] : p.agent_mask, gm);
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Split-K form for a few row tiles (64 < M <= 512: the tokens of a short turn).  A block of the kernel
// above needs about 0.4 us per 64-deep k-block whatever its tile width, so the whole K extent costs one
// block 25 us at d_model 4096 even when there is almost no work.  Here the K extent of one 128 x BN tile is
// divided over the KS = 3 ... 8 blocks of a cluster (grid = (KS, column tiles, row tiles)); each block accumulates its
// K slice in TMEM exactly as above, writes the fp32 accumulator into its own shared memory (over the ring,
// which is idle by then), and after a cluster barrier block r adds up columns [r*cw, (r+1)*cw) of all KS
// partial tiles over distributed shared memory — in rank order, so the result does not depend on timing —
// and routes them to the caches with the same epilogue.  No rotary epilogue here (a head's two halves would
// have to land in one block's slice); rotary calls use the kernel above.
__global__ void __launch_bounds__(GEMM_THREADS, 2)
proj_gemm_splitk_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GemmParams p) {
  // The declared alignment places the dynamic shared memory on a 1024-byte boundary (the swizzle atoms need it and
  // the peers' addresses must correspond).  Should the base ever be unaligned, every block of the grid says so and leaves.
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw;
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicOr(p.status, StatusBits::TIMEOUT);
    return;
  }
  const int b_bytes = p.BN * GEMM_BK * 2;
  const int stage_bytes = GEMM_A_BYTES + b_bytes;
  // The dumped accumulator is laid out slice by slice: block r of the cluster will reduce columns
  // [r*cw, (r+1)*cw), and finds them in every peer as one block of 128 rows x (cw + 4) floats (the 4 floats
  // of padding keep the row-per-thread dump free of bank conflicts), which it can read with consecutive lanes
  // on consecutive 16-byte pieces.
  const int cw = (((p.BN + (int)gridDim.x - 1) / (int)gridDim.x) + 7) / 8 * 8;   // columns reduced by one block (a multiple of 8)
  const int XS = cw + 4;                                        // row stride (floats) inside a slice
  const int ring_bytes = p.stages * stage_bytes, dump_bytes = (int)gridDim.x * GEMM_BM * XS * 4;
  const int data_bytes = ((ring_bytes > dump_bytes ? ring_bytes : dump_bytes) + 1023) & ~1023;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + data_bytes);
  // barrier map: full[stages] | empty[stages] | acc_full
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = full0 + 8 * p.stages;
  const uint32_t acc_full = empty0 + 8 * p.stages;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KS = gridDim.x, rank = blockIdx.x;                  // the cluster spans grid.x
  const int nkb = p.K / GEMM_BK;                                // K slices need not be equal (KS = 3, 5, 6, 7 are allowed):
  const int kb0 = (rank * nkb) / KS;                            // slice r = [r nkb / KS, (r+1) nkb / KS), each at least
  const int nkb_s = ((rank + 1) * nkb) / KS - kb0;              // floor(nkb / KS) >= 2 k-blocks (the host sees to that)
  const int m0 = blockIdx.z * GEMM_BM, n0 = blockIdx.y * p.BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    // the ring's first fill is requested right away (this thread is the producer): its latency then overlaps the
    // tensor-memory allocation and the block barrier below
    for (int it = 0; it < min(p.stages, nkb_s); ++it) {
      const uint32_t sa = smem_u32(smem + (size_t)it * stage_bytes);
      mbar_expect_tx(full0 + 8 * it, stage_bytes);
      tma_load_2d(sa, &map_x, (kb0 + it) * GEMM_BK, m0, full0 + 8 * it);
      tma_load_3d(sa + GEMM_A_BYTES, &map_w, 0, n0, kb0 + it, full0 + 8 * it);
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_holder)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    if (lane == 0) {
      for (int it = p.stages; it < nkb_s; ++it) {          // the first fill was issued above
        const int s = it % p.stages;
        mbar_wait(empty0 + 8 * s, ((it / p.stages) - 1) & 1, p.status);
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        mbar_expect_tx(full0 + 8 * s, stage_bytes);
        tma_load_2d(sa, &map_x, (kb0 + it) * GEMM_BK, m0, full0 + 8 * s);
        tma_load_3d(sa + GEMM_A_BYTES, &map_w, 0, n0, kb0 + it, full0 + 8 * s);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(p.BN);
      const uint64_t da0 = umma_desc_sw128(smem_u32(smem));
      const uint64_t db0 = umma_desc_sw128(smem_u32(smem) + GEMM_A_BYTES);
      for (int it = 0; it < nkb_s; ++it) {
        const int s = it % p.stages;
        mbar_wait(full0 + 8 * s, (it / p.stages) & 1, p.status);
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint64_t so = (uint64_t)((s * stage_bytes) >> 4);
#pragma unroll
        for (int k = 0; k < GEMM_BK / 16; ++k)
          umma_bf16(tmem_base, da0 + so + 2 * k, db0 + so + 2 * k, idesc, (it | k) ? 1u : 0u);
        umma_commit(empty0 + 8 * s);
      }
      umma_commit(acc_full);                       // every MMA of the slice has completed: the ring is idle too
    }
  } else {
    // ---- this block's partial tile: TMEM (lane = row) -> shared memory, fp32 [128][XS]
    const int lane_base = (warp & 3) * 32;
    const int row = lane_base + lane;
    float* dump = reinterpret_cast<float*>(smem);
    mbar_wait(acc_full, 0, p.status);
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    for (int c0 = 0; c0 < p.BN; c0 += 16) {
      uint32_t r[16];
      tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_base) << 16) + c0, r);
      asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
      for (int k = 0; k < 16; k += 4) {
        const int c = c0 + k, sl = c / cw;
        *reinterpret_cast<uint4*>(dump + ((size_t)sl * GEMM_BM + row) * XS + (c - sl * cw)) = make_uint4(r[k], r[k + 1], r[k + 2], r[k + 3]);
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  }
  // every block's partial tile is complete and visible
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  {
    const int t = threadIdx.x;                                  // the producer and MMA warps help with the merge
    switch (KS) {
      case 8: splitk_reduce<8>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
      case 7: splitk_reduce<7>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
      case 6: splitk_reduce<6>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
      case 5: splitk_reduce<5>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
      case 4: splitk_reduce<4>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
      case 3: splitk_reduce<3>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
      default: splitk_reduce<2>(p, smem_u32(smem), rank, cw, m0, n0, t); break;
    }
  }
  // nobody leaves while a peer may still read its partial tile
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Split-K with a merge by bulk sends (clusters of 2 .. 4 blocks: the turns of a few hundred to a thousand rows).
// Same main loop as the kernel above.  Then block r dumps the column slices it does NOT own to shared memory
// (over the idle ring), tells its peers that its ring is idle, and - once every peer has said the same - sends
// slice j to block j with ONE cp.async.bulk (shared::cta -> shared::cluster), which counts the bytes on an
// mbarrier of the receiver.  A receiver waits for its (KS - 1) slices, adds them to its own slice (re-read from
// tensor memory) in rank order - the order of the pulling kernel, bit for bit - and stores through the same
// epilogue routing.  The copy engine moves a slice (32 .. 66 KB) in well under a microsecond, where sixteen
// 16-byte loads per thread over distributed shared memory moved the same bytes in 4 .. 6 us.
// Shared memory: [ring | overlaid: dump of KS-1 slices, then receive area of KS-1 slices] [barriers].
// Finer splits (GemmParams::direct_send; twice KS-1 slices would not fit): no dump at all - every epilogue thread
// sends the 16-byte pieces of its row straight from registers (st.async.v4 into the owner's receive area, which
// alone overlays the ring), only the rows of the tile that exist; no barrier at the end either, since a send
// carries its data with it.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}

// What the routing of a row's 16-byte pieces needs to know about the row, worked out once (no rotary keys here).
struct RowRoute {
  bool ok;
  long long slot, slot2, base_row;
  unsigned long long mask;
  __device__ __forceinline__ void init(const GemmParams& p, int gm) {
    ok = gm < p.M;
    slot = 0; slot2 = -1;
    if (ok) {
      slot = p.slot_mapping ? (long long)p.slot_mapping[gm] : p.start_slot + gm;
      if (slot < 0 || slot >= p.n_blocks * PAGE) { atomicOr(p.status, StatusBits::BAD_INDEX); ok = false; slot = 0; }
    }
    mask = (p.row_masks && ok) ? p.row_masks[gm] : p.agent_mask;
    if (p.lr_copy_slots && ok) {
      slot2 = p.lr_copy_slots[gm];
      if (slot2 >= p.n_blocks * PAGE) { atomicOr(p.status, StatusBits::BAD_INDEX); slot2 = -1; }
    }
    base_row = (((slot / PAGE) * p.n_kv * PAGE) + (slot % PAGE)) << p.hd_shift;
  }
  // columns gc .. gc + 7 of the call's output (gc is the same in every lane: the branches are warp-uniform)
  __device__ __forceinline__ void store8(const GemmParams& p, int gc, const float (&v8)[8]) const {
    if (!ok) return;
    const int hs = p.hd_shift, w = p.n_kv << hs;
    uint4 v;
    v.x = pack_bf16(v8[0], v8[1]); v.y = pack_bf16(v8[2], v8[3]); v.z = pack_bf16(v8[4], v8[5]); v.w = pack_bf16(v8[6], v8[7]);
    if (p.mode == 1 || (p.mode == 2 && gc < 2 * w)) {
      const bool is_v = gc >= w;
      const int cc = is_v ? gc - w : gc;
      const int g = cc >> hs, c = cc & (p.hd - 1);
      *reinterpret_cast<uint4*>((is_v ? p.base_v : p.base_k) + base_row + ((long long)(g * PAGE) << hs) + c) = v;
    } else {
      const int n_lrk = p.rank_k > 0 ? (p.n_agents << p.rk_shift) : 0;
      const int gl = p.mode == 2 ? gc - 2 * w : gc;
      const bool is_v = gl >= n_lrk;
      const int sh = is_v ? p.rv_shift : p.rk_shift;
      const int cc = is_v ? gl - n_lrk : gl;
      const int agent = cc >> sh, ri = cc & ((1 << sh) - 1);
      if (!((mask >> agent) & 1ull)) return;
      __nv_bfloat16* arr = (is_v ? p.lr_v : p.lr_k) + (((long long)agent * p.n_blocks * PAGE) << sh) + ri;
      *reinterpret_cast<uint4*>(arr + (slot << sh)) = v;
      if (slot2 >= 0) *reinterpret_cast<uint4*>(arr + (slot2 << sh)) = v;
    }
  }
};

__global__ void __launch_bounds__(GEMM_THREADS, 1)
proj_gemm_splitk_push_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GemmParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw;
  if ((smem_u32(smem_raw) & 1023u) != 0) {               // the peers' addresses must correspond
    if (threadIdx.x == 0) atomicOr(p.status, StatusBits::TIMEOUT);
    return;
  }
  const int KS = gridDim.x, rank = blockIdx.x;           // the cluster spans grid.x
  const int b_bytes = p.BN * GEMM_BK * 2;
  const int stage_bytes = GEMM_A_BYTES + b_bytes;
  const int cw = (((p.BN + KS - 1) / KS) + 7) / 8 * 8;   // columns finished by one block (a multiple of 8)
  const int XS = cw + 4;                                 // row stride (floats) inside a slice: conflict-free row-per-thread access
  const int slice_bytes = GEMM_BM * XS * 4;              // a multiple of 16
  const bool direct = p.direct_send != 0;               // the same in every block
  const int ring_bytes = p.stages * stage_bytes, merge_bytes = (direct ? 1 : 2) * (KS - 1) * slice_bytes;
  const int data_bytes = ((ring_bytes > merge_bytes ? ring_bytes : merge_bytes) + 1023) & ~1023;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + data_bytes);
  // barrier map: full[stages] | empty[stages] | acc_full | ready (peers whose ring is idle) | recv (bytes received)
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = full0 + 8 * p.stages;
  const uint32_t acc_full = empty0 + 8 * p.stages;
  const uint32_t ready_bar = acc_full + 8, recv_bar = acc_full + 16;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 4);
  float* dump = reinterpret_cast<float*>(smem);                                       // [KS-1][128][XS]
  float* recv = reinterpret_cast<float*>(smem + (direct ? (size_t)0 : (size_t)(KS - 1) * slice_bytes));   // [KS-1][128][XS]
  const int rows_valid = min(GEMM_BM, p.M - blockIdx.z * GEMM_BM);                     // rows of this tile that exist
  const int vw_own = max(0, min(cw, p.BN - rank * cw));                                // columns of this block's slice that exist

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb = p.K / GEMM_BK;
  const int kb0 = (rank * nkb) / KS;
  const int nkb_s = ((rank + 1) * nkb) / KS - kb0;
  const int m0 = blockIdx.z * GEMM_BM, n0 = blockIdx.y * p.BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(acc_full, 1);
    mbar_init(ready_bar, KS - 1);
    mbar_init(recv_bar, 1);
    // the one arrival, and the bytes to come: whole slices by bulk copy, or the existing rows and columns piece by piece
    mbar_expect_tx(recv_bar, direct ? (uint32_t)((KS - 1) * rows_valid * vw_own * 4) : (uint32_t)((KS - 1) * slice_bytes));
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    for (int it = 0; it < min(p.stages, nkb_s); ++it) {
      const uint32_t sa = smem_u32(smem + (size_t)it * stage_bytes);
      mbar_expect_tx(full0 + 8 * it, stage_bytes);
      tma_load_2d(sa, &map_x, (kb0 + it) * GEMM_BK, m0, full0 + 8 * it);
      tma_load_3d(sa + GEMM_A_BYTES, &map_w, 0, n0, kb0 + it, full0 + 8 * it);
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_holder)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;
  // every block's barriers exist before anybody arrives on them from outside (the wait comes with the first remote use)
  asm volatile("barrier.cluster.arrive.relaxed.aligned;\n" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      for (int it = p.stages; it < nkb_s; ++it) {
        const int s = it % p.stages;
        mbar_wait(empty0 + 8 * s, ((it / p.stages) - 1) & 1, p.status);
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        mbar_expect_tx(full0 + 8 * s, stage_bytes);
        tma_load_2d(sa, &map_x, (kb0 + it) * GEMM_BK, m0, full0 + 8 * s);
        tma_load_3d(sa + GEMM_A_BYTES, &map_w, 0, n0, kb0 + it, full0 + 8 * s);
      }
    }
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(p.BN);
      const uint64_t da0 = umma_desc_sw128(smem_u32(smem));
      const uint64_t db0 = umma_desc_sw128(smem_u32(smem) + GEMM_A_BYTES);
      for (int it = 0; it < nkb_s; ++it) {
        const int s = it % p.stages;
        mbar_wait(full0 + 8 * s, (it / p.stages) & 1, p.status);
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint64_t so = (uint64_t)((s * stage_bytes) >> 4);
#pragma unroll
        for (int k = 0; k < GEMM_BK / 16; ++k)
          umma_bf16(tmem_base, da0 + so + 2 * k, db0 + so + 2 * k, idesc, (it | k) ? 1u : 0u);
        umma_commit(empty0 + 8 * s);
      }
      umma_commit(acc_full);                       // every MMA of the slice has completed: the ring is idle too
    }
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  } else {
    const int lane_base = (warp & 3) * 32;
    const int row = lane_base + lane;
    const int et = threadIdx.x - 64;                // 0 .. 127 among the four epilogue warps
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");   // the peers' barriers are initialised
    mbar_wait(acc_full, 0, p.status);
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    // this block's ring is idle: the peers may send into the receive area that overlays it
    if (et < KS - 1) {
      const int peer = et < rank ? et : et + 1;
      uint32_t remote;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote) : "r"(ready_bar), "r"(peer));
      asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(remote) : "memory");
    }
    RowRoute route;
    route.init(p, m0 + row);
    const uint32_t trow = tmem_base + (static_cast<uint32_t>(lane_base) << 16);
    // ---- the peers' slices, one after the other: TMEM (lane = row) -> shared memory fp32 [slot][128][XS] (slot = the
    //      peer's rank with the own rank left out), then one bulk copy into the peer's receive area while the next
    //      slice is being dumped
    if (direct) mbar_wait_cluster(ready_bar, 0, p.status);           // every peer's ring is idle
    for (int k = 1; direct && k < KS; ++k) {
      const int sl = rank + k < KS ? rank + k : rank + k - KS;
      const int c_lo = sl * cw, vw = min(cw, p.BN - c_lo);
      // this row of slice sl goes to slot (own rank, sl's rank left out) of block sl's receive area
      const uint32_t dst_local = smem_u32(recv) + (uint32_t)((((rank < sl ? rank : rank - 1) * GEMM_BM + row) * XS) * 4);
      const uint32_t dst = dsmem_addr(dst_local, sl), bar = dsmem_addr(recv_bar, sl);
      const bool live = row < rows_valid;
      int c = 0;
      for (; c + 32 <= vw; c += 32) {
        uint32_t r0[16], r1[16];
        tmem_ld16(trow + c_lo + c, r0);
        tmem_ld16(trow + c_lo + c + 16, r1);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
        if (live) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            st_async_b32x4(dst + (c + 4 * q) * 4, r0[4 * q], r0[4 * q + 1], r0[4 * q + 2], r0[4 * q + 3], bar);
            st_async_b32x4(dst + (c + 16 + 4 * q) * 4, r1[4 * q], r1[4 * q + 1], r1[4 * q + 2], r1[4 * q + 3], bar);
          }
        }
      }
      for (; c + 8 <= vw; c += 8) {
        uint32_t r[8];
        tmem_ld8(trow + c_lo + c, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
        if (live) {
          st_async_b32x4(dst + c * 4, r[0], r[1], r[2], r[3], bar);
          st_async_b32x4(dst + (c + 4) * 4, r[4], r[5], r[6], r[7], bar);
        }
      }
    }
    for (int k = 1; !direct && k < KS; ++k) {
      const int sl = rank + k < KS ? rank + k : rank + k - KS;
      const int c_lo = sl * cw, vw = min(cw, p.BN - c_lo);           // valid width of the slice (a multiple of 8, may be <= 0)
      float* drow = dump + ((size_t)(sl < rank ? sl : sl - 1) * GEMM_BM + row) * XS;
      int c = 0;
      for (; c + 32 <= vw; c += 32) {
        uint32_t r0[16], r1[16];
        tmem_ld16(trow + c_lo + c, r0);
        tmem_ld16(trow + c_lo + c + 16, r1);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          *reinterpret_cast<uint4*>(drow + c + 4 * q) = make_uint4(r0[4 * q], r0[4 * q + 1], r0[4 * q + 2], r0[4 * q + 3]);
          *reinterpret_cast<uint4*>(drow + c + 16 + 4 * q) = make_uint4(r1[4 * q], r1[4 * q + 1], r1[4 * q + 2], r1[4 * q + 3]);
        }
      }
      for (; c + 8 <= vw; c += 8) {
        uint32_t r[8];
        tmem_ld8(trow + c_lo + c, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
        *reinterpret_cast<uint4*>(drow + c) = make_uint4(r[0], r[1], r[2], r[3]);
        *reinterpret_cast<uint4*>(drow + c + 4) = make_uint4(r[4], r[5], r[6], r[7]);
      }
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");         // the copy engine reads what these threads wrote
      asm volatile("bar.sync 1, 128;\n" ::: "memory");                       // the four epilogue warps
      if (et == 0) {
        if (k == 1) mbar_wait_cluster(ready_bar, 0, p.status);                // every peer's ring is idle
        // slice sl of this block goes to slot (own rank, sl's rank left out) of block sl's receive area
        const uint32_t src = smem_u32(dump) + (uint32_t)((sl < rank ? sl : sl - 1) * slice_bytes);
        const uint32_t dst_local = smem_u32(recv) + (uint32_t)((rank < sl ? rank : rank - 1) * slice_bytes);
        uint32_t dst, bar;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(dst) : "r"(dst_local), "r"(sl));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(bar) : "r"(recv_bar), "r"(sl));
        asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                     ::"r"(dst), "r"(src), "r"(slice_bytes), "r"(bar) : "memory");
      }
    }
    // ---- own slice (tensor memory) + received slices, in rank order, routed to the caches
    mbar_wait_cluster(recv_bar, 0, p.status);
    {
      const int c_lo = rank * cw, vw = min(cw, p.BN - c_lo);
      const bool wide = KS <= GEMM_PUSH_MAX_KS;         // 16 columns at a time while the peers' pieces fit in registers
      for (int c = 0; c + 8 <= vw; c += wide ? 16 : 8) {
        const bool two = wide && c + 16 <= vw;          // 8 at a ragged end (the same in every lane)
        uint32_t own[16];
        if (two) {
          tmem_ld16(trow + c_lo + c, own);
        } else {
          uint32_t o8[8];
          tmem_ld8(trow + c_lo + c, o8);
#pragma unroll
          for (int q = 0; q < 8; ++q) { own[q] = o8[q]; own[8 + q] = 0u; }
        }
        float4 pr[GEMM_MAX_KS - 1][4];
#pragma unroll
        for (int j = 0; j < GEMM_MAX_KS - 1; ++j) {
          if (j < KS - 1) {
            const float* src = recv + ((size_t)j * GEMM_BM + row) * XS + c;
            pr[j][0] = *reinterpret_cast<const float4*>(src);
            pr[j][1] = *reinterpret_cast<const float4*>(src + 4);
            if (j < GEMM_PUSH_MAX_KS - 1) {
              if (two) { pr[j][2] = *reinterpret_cast<const float4*>(src + 8); pr[j][3] = *reinterpret_cast<const float4*>(src + 12); }
            }
          }
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h == 1 && !two) break;
          float v8[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) v8[q] = 0.f;
          // rank order: slot j of the receive area holds rank j (j < own rank) or j + 1, so the own slice goes in
          // just before slot `rank` (or last)
          auto add_own = [&]() {
#pragma unroll
            for (int q = 0; q < 8; ++q) v8[q] += __uint_as_float(own[8 * h + q]);
          };
#pragma unroll
          for (int j = 0; j < GEMM_MAX_KS - 1; ++j) {
            if (j < KS - 1 && (h == 0 || j < GEMM_PUSH_MAX_KS - 1)) {
              if (j == rank) add_own();
              const float4 a = pr[j][h == 0 ? 0 : 2], b = pr[j][h == 0 ? 1 : 3];
              v8[0] += a.x; v8[1] += a.y; v8[2] += a.z; v8[3] += a.w; v8[4] += b.x; v8[5] += b.y; v8[6] += b.z; v8[7] += b.w;
            }
          }
          if (rank == KS - 1) add_own();
          const int gc = n0 + c_lo + c + 8 * h;
          if (gc < p.N_out) route.store8(p, gc, v8);
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  }
  // Bulk sends read the sender's shared memory: nobody leaves before every block has received everything.  Direct
  // sends carry their data with them, and a receiver stays until it has everything: no barrier.
  __syncwarp();
  if (!direct) {
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

}  // namespace precc
