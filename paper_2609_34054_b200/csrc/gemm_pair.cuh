// The projection GEMM with two SMs per output tile (tcgen05 cta_group::2).
//
// A block pair (a cluster of two) owns a 256 x BN output tile.  Each block stages ITS 128 rows of X and ITS half of
// the weight tile (BN/2 weight rows) per 64-deep k-block; one thread of the pair's first block issues
// tcgen05.mma.cta_group::2, which multiplies the 256 rows held by the two blocks with the BN weight rows held by
// the two blocks and leaves rows 0..127 of the result in the first block's tensor memory and rows 128..255 in the
// second's.  Per block and k-block that is 16 KB + BN/2 x 128 B written to and read from shared memory instead of
// 16 KB + BN x 128 B: the one-block kernel is bound by exactly that traffic (MMA operand reads plus the ring's own
// fills exceed what shared memory delivers), the pair is not.
//
// Hand-offs inside the pair:
//   full[s]     first block's barrier; the TMA copies of BOTH blocks complete their bytes on it (.cta_group::2
//               copies may signal the peer's barrier), the first block's producer arms it with the pair's byte count
//   empty[s]    one barrier in each block, signalled together by the issuing thread's tcgen05.commit (multicast to
//               the pair): the stage of both blocks may be refilled once the MMAs have read it
//   acc_full    likewise one in each block: the accumulator of a tile is complete, both epilogues may read
//   acc_empty   first block's barrier, 8 arrivals: the four epilogue warps of either block have drained the buffer
// No copy is a multicast copy: every block fetches its own operands.  Every wait is bounded (see mbar_wait); the
// cluster barrier before the exit keeps a block alive while its peer may still signal or read it.
#pragma once
#include "gemm_tc.cuh"

namespace precc {

constexpr int GEMM_PAIR_BM = 2 * GEMM_BM;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
// TMA copies of a block pair: the bytes are counted on `bar`, which may live in the peer block (no multicast).
__device__ __forceinline__ void tma_pair_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_pair_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// Instruction descriptor of the pair MMA: D fp32, A/B bf16, both K-major, M = 256 (two blocks), N = n.
__device__ __forceinline__ uint32_t umma_pair_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(GEMM_PAIR_BM >> 4) << 24);
}
__device__ __forceinline__ void umma_pair_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
// Completion of the pair's MMAs issued so far, signalled on the barrier at this offset in both blocks.
__device__ __forceinline__ void umma_pair_commit_both(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n"
               ::"r"(bar), "h"(both) : "memory");
}
__device__ __forceinline__ void pair_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
proj_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the 128-byte swizzle atoms (the same offset in both blocks: the dynamic shared memory
  // of the two starts at the same address in each block's window)
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int half_n = p.BN / 2;                           // weight rows staged by each block
  const int b_bytes = half_n * GEMM_BK * 2;
  const int stage_bytes = GEMM_A_BYTES + b_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes);
  // barrier map (the same in both blocks): full[stages] | empty[stages] | acc_full[2] | acc_empty[2]
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = full0 + 8 * p.stages;
  const uint32_t acc_full = empty0 + 8 * p.stages;
  const uint32_t acc_empty = acc_full + 16;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0: issues the MMAs and owns full / acc_empty
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int nkb = p.K / GEMM_BK;
  const int n_tiles_n = (p.N_out + p.BN - 1) / p.BN;
  // Row tiles of 256 rows.  With a single column tile and more tiles than pairs the count is rounded up to a multiple
  // of the pairs and the tiles are spread evenly over the rows (neighbours overlap by a few rows, computed twice
  // with identical results), so that every pair streams the same number of rows.
  const int m_plain = (p.M + GEMM_PAIR_BM - 1) / GEMM_PAIR_BM;
  const bool spread = p.spread_rows && n_tiles_n == 1 && m_plain > n_pairs && p.M >= GEMM_PAIR_BM;
  const int m_tiles = spread ? ((m_plain + n_pairs - 1) / n_pairs) * n_pairs : m_plain;
  const int n_tiles = m_tiles * n_tiles_n;
  auto row0_of = [&](int mt) -> int {
    if (!spread) return mt * GEMM_PAIR_BM;
    return (int)(((long long)mt * (p.M - GEMM_PAIR_BM)) / (m_tiles - 1));   // first tile at 0, last one ends at M
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(acc_full, 1); mbar_init(acc_full + 8, 1);
    mbar_init(acc_empty, 8); mbar_init(acc_empty + 8, 8);         // four epilogue warps in each of the two blocks
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_holder)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  pair_sync();                                           // the peer's barriers exist before anything signals them
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    if (lane == 0) {
      // producer: this block's rows of X and its half of the weight tile; bytes are counted on the first block's barrier
      const uint32_t full0_lead = map_to_rank(full0, 0);
      int it = 0;
      for (int t = pair; t < n_tiles; t += n_pairs) {
        const int m0 = row0_of(t / n_tiles_n) + (int)rank * GEMM_BM, n0 = (t % n_tiles_n) * p.BN + (int)rank * half_n;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % p.stages;
          if (it >= p.stages) mbar_wait(empty0 + 8 * s, ((it / p.stages) - 1) & 1, p.status);
          GEMM_STAMP(p, it, 0);
          const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
          if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * stage_bytes);
          tma_pair_load_2d(sa, &map_x, kb * GEMM_BK, m0, full0_lead + 8 * s);
          tma_pair_load_3d(sa + GEMM_A_BYTES, &map_w, 0, n0, kb, full0_lead + 8 * s);      // packed weights are k-blocked
          GEMM_STAMP(p, it, 1);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_pair_idesc_bf16(p.BN);
      const uint64_t da0 = umma_desc_sw128(smem_u32(smem));
      const uint64_t db0 = umma_desc_sw128(smem_u32(smem) + GEMM_A_BYTES);
      int it = 0, i = 0;
      for (int t = pair; t < n_tiles; t += n_pairs, ++i) {
        const int buf = i & 1;
        if (i >= 2) mbar_wait(acc_empty + 8 * buf, ((i >> 1) - 1) & 1, p.status);   // both epilogues have drained this buffer
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
            umma_pair_bf16(d, da0 + so + 2 * k, db0 + so + 2 * k, idesc, (kb | k) ? 1u : 0u);
          GEMM_STAMP(p, it, 3);
          umma_pair_commit_both(empty0 + 8 * s);   // the stage of both blocks is reusable once these MMAs have read it
          GEMM_STAMP(p, it, 4);
        }
        umma_pair_commit_both(acc_full + 8 * buf); // accumulator of this tile complete in both blocks
      }
    }
  } else {
    // ---- epilogue: this block's 128 rows of the tile; TMEM lane = row; this warp may touch lanes 32*(warp%4) .. +31
    const int lane_base = (warp & 3) * 32;
    const uint32_t acc_empty_lead = map_to_rank(acc_empty, 0);
    int i = 0;
    for (int t = pair; t < n_tiles; t += n_pairs, ++i) {
      const int buf = i & 1;
      const int m0 = row0_of(t / n_tiles_n) + (int)rank * GEMM_BM, n0 = (t % n_tiles_n) * p.BN;
      gemm_epilogue_tile(p, tmem_base + buf * p.BN, m0, n0, lane_base, lane, acc_full + 8 * buf, (i >> 1) & 1);
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(acc_empty_lead + 8 * buf) : "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  pair_sync();                                           // nobody leaves while the peer may still signal or read this block
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

}  // namespace precc
