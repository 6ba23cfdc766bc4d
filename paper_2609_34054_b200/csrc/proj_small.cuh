// Projection for a handful of rows (decode steps, M <= 64): Y[M x n_out] = X[M x K] . Wt^T with the same
// routing epilogue as the tensor-memory GEMM (LR caches, base caches, or both).
//
// With M this small the work is one pass over the packed weights (n_out x K bf16), so the kernel is a
// weight-streaming kernel: HBM-bound at n_out*K*2 bytes.  A 128-row tcgen05 tile would leave all but
// n_out/BN blocks idle; here the grid covers every SM:
//   block  = 64 output columns (128 when M > 16) x one K slice; the K slices of a column group form a
//            thread-block cluster (split-K, up to 8);
//   loads  = TMA: per 64-deep k step one box of W rows (contiguous in memory: the packed weights are
//            k-blocked, [K/64][n_out][64]) and one box of X rows (rows past M are zero-filled
//            by the out-of-bounds rule) into a 4-slot ring of 128-byte-swizzled shared memory, issued by
//            a producer warp (full/empty mbarriers).  The ring is kept small on purpose: every cluster of
//            the grid must be resident at once, or the launch runs in two waves;
//   math   = mma.sync m16n8k16 (bf16 -> fp32): X rows on the M axis, a warp owns 8 (16 when M > 16)
//            output columns; fragments come from shared memory with ldmatrix;
//   reduce = every block finishes one slice of its group's columns.  The consumer threads SEND their accumulator
//            pairs to the block that owns the column (st.async into the owner's shared memory, bytes counted on
//            the owner's mbarrier); the owner waits for its byte count, adds the partials in rank order
//            (deterministic) and scatters bf16 pieces into the paged caches.  No global scratch, no atomics, and
//            no cluster barrier on the critical path (one, relaxed, at the start makes the mbarriers visible).
//            Rotary keys keep the earlier form: partial tiles in shared memory, a cluster barrier, and each block
//            reads its slice - and the partner half of a head - from its peers over distributed shared memory.
// Rotary keys (GemmParams::rope): the reducing thread of the lower half of a head also gathers the partner
// piece hd/2 columns further and writes both rotated; the block tile therefore holds whole heads.
// The K split depends on K alone, so an output value does not depend on which entry point, which other
// columns or how many other rows were in the call.
#pragma once
#include "gemm_tc.cuh"

namespace precc {

constexpr int PS_WARPS = 8;
constexpr int PS_BK = 64;                   // k elements per step: one 128-byte swizzle row
constexpr int PS_MAX_M = 64;
constexpr int PS_STAGES = 4;
constexpr int PS_THREADS = (PS_WARPS + 1) * 32;       // consumer warps + one producer warp
__host__ __device__ constexpr int ps_nt(int mt) { return mt > 1 ? 2 : 1; }               // 8-column n-tiles per warp
__host__ __device__ constexpr int ps_cols(int mt) { return PS_WARPS * 8 * ps_nt(mt); }   // output columns per block
__host__ __device__ constexpr int ps_step_bytes(int mt) { return (ps_cols(mt) + mt * 16) * PS_BK * 2; }
__host__ __device__ constexpr int ps_recv_bytes(int mt) { return mt * 16 * ps_cols(mt) * 4; }   // [cluster rank][row][own columns] fp32
__host__ __device__ constexpr int ps_smem_bytes(int mt) {
  return PS_STAGES * ps_step_bytes(mt) + 128 + ps_recv_bytes(mt) + 1024;   // ring | mbarriers | receive area | alignment slack
}

template <int MT>
__global__ void __launch_bounds__(PS_THREADS)
proj_small_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GemmParams p,
                  const int k_slice) {
  constexpr int NT = ps_nt(MT);
  constexpr int COLS = ps_cols(MT);
  constexpr int W_BYTES = COLS * PS_BK * 2;
  constexpr int STEP_BYTES = ps_step_bytes(MT);
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint32_t rank, CS;
  asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(rank));
  asm volatile("mov.u32 %0, %%cluster_nctaid.x;\n" : "=r"(CS));
  const int group = blockIdx.x / CS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k0 = rank * k_slice;
  const int steps = k_slice / PS_BK;
  const uint32_t tiles = smem_u32(smem);
  const uint32_t full0 = tiles + PS_STAGES * STEP_BYTES, empty0 = full0 + 8 * PS_STAGES;
  const uint32_t recv_bar = empty0 + 8 * PS_STAGES;
  const uint32_t recv_u32 = full0 + 128;                // behind the barriers; never overlaid: peers send while this block computes
  const bool push = !p.rope;                            // the same in every block of the grid
  const int cpb = COLS / CS;                            // columns finished by one block (a power of two >= 8)

  if (threadIdx.x == 0) {
    for (int s = 0; s < PS_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, PS_WARPS); }
    mbar_init(recv_bar, 1);
    if (push) mbar_expect_tx(recv_bar, (uint32_t)(CS * p.M * cpb * 4));   // the one arrival, and the bytes to come: rows < M of every peer
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  }
  __syncthreads();
  if (push) asm volatile("barrier.cluster.arrive.relaxed.aligned;\n" ::: "memory");   // waited for before the first send
  // The weights are not the preceding kernel's to write: the first ring fill of W boxes is requested before the wait
  // for that kernel (programmatic dependent launch), so a block that is resident early has them in shared memory
  // when its predecessor ends.  X (the previous kernel's output) and every store stay behind the wait.
  const int pre = steps < PS_STAGES ? steps : PS_STAGES;
  if (warp == PS_WARPS && lane == 0) {
    for (int s = 0; s < pre; ++s) {
      mbar_expect_tx(full0 + 8 * s, STEP_BYTES);
      tma_load_3d(tiles + s * STEP_BYTES, &map_w, 0, group * COLS, k0 / PS_BK + s, full0 + 8 * s);
    }
  }
  pdl_wait();                 // X may be the previous kernel's output; the caches may still be read by it
  pdl_launch_dependents();

  float acc[MT][NT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int t = 0; t < NT; ++t) { acc[mt][t][0] = acc[mt][t][1] = acc[mt][t][2] = acc[mt][t][3] = 0.f; }

  if (warp == PS_WARPS) {
    // ---- producer: one lane walks the k steps of this block's slice
    if (lane == 0) {
      for (int s = 0; s < pre; ++s)                      // the X boxes of the steps whose W boxes are already on their way
        tma_load_2d(tiles + s * STEP_BYTES + W_BYTES, &map_x, k0 + s * PS_BK, 0, full0 + 8 * s);
      for (int s = pre; s < steps; ++s) {
        const int slot = s % PS_STAGES;
        mbar_wait(empty0 + 8 * slot, ((s / PS_STAGES) - 1) & 1, p.status);
        const uint32_t dst = tiles + slot * STEP_BYTES;
        mbar_expect_tx(full0 + 8 * slot, STEP_BYTES);
        tma_load_3d(dst, &map_w, 0, group * COLS, k0 / PS_BK + s, full0 + 8 * slot);   // one contiguous run of the k-blocked weights
        tma_load_2d(dst + W_BYTES, &map_x, k0 + s * PS_BK, 0, full0 + 8 * slot);
      }
    }
  } else {
    const int mi = lane >> 3, ri = lane & 7;
    for (int s = 0; s < steps; ++s) {
      const int slot = s % PS_STAGES;
      mbar_wait(full0 + 8 * slot, (s / PS_STAGES) & 1, p.status);
      const uint32_t wt = tiles + slot * STEP_BYTES, xt = wt + W_BYTES;
#pragma unroll
      for (int j = 0; j < 2; ++j) {                      // two k steps of 16 per ldmatrix of W
        uint32_t b[NT][4];
#pragma unroll
        for (int t = 0; t < NT; ++t) ldsm_x4(b[t], wt + swz_off<8>((warp * NT + t) * 8 + ri, 4 * j + mi));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t a[4];
            ldsm_x4(a, xt + swz_off<8>(mt * 16 + ri + (mi & 1) * 8, 2 * (2 * j + h) + (mi >> 1)));
#pragma unroll
            for (int t = 0; t < NT; ++t) mma_bf16_16816(acc[mt][t], a, b[t][2 * h], b[t][2 * h + 1]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(empty0 + 8 * slot) : "memory");
    }
  }
  if (push) {
    // ---- merge by sends: accumulator pairs go straight from registers to the owner of their column
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");   // every peer's mbarrier is initialised (long since)
    const int cshift = 31 - __clz(cpb);
    if (warp < PS_WARPS) {
      const int r = lane >> 2, q = lane & 3;
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          const int col = (warp * NT + t) * 8 + 2 * q;
          const int owner = col >> cshift;
          const uint32_t bar = dsmem_addr(recv_bar, owner);
          const uint32_t dst = recv_u32 + (uint32_t)(((rank * (MT * 16) + mt * 16 + r) * cpb + (col & (cpb - 1))) * 4);
          if (mt * 16 + r < p.M) st_async_f32x2(dsmem_addr(dst, owner), acc[mt][t][0], acc[mt][t][1], bar);
          if (mt * 16 + r + 8 < p.M) st_async_f32x2(dsmem_addr(dst + 8 * cpb * 4, owner), acc[mt][t][2], acc[mt][t][3], bar);
        }
    }
    // ---- this block finishes columns [rank*cpb, (rank+1)*cpb) of its group: 8-column pieces, partials added in rank order
    const int ppr = cpb / 8;
    const int n_items = p.M * ppr;
    int it = threadIdx.x;
    int row = it / ppr, pc = it - row * ppr;              // worked out before the wait
    mbar_wait_cluster(recv_bar, 0, p.status);
    const float* recv = reinterpret_cast<const float*>(smem + PS_STAGES * STEP_BYTES + 128);
    for (; it < n_items; it += PS_THREADS, row = it / ppr, pc = it - row * ppr) {
      const int gc = group * COLS + rank * cpb + pc * 8;
      if (gc >= p.N_out) continue;
      long long slot = p.slot_mapping ? (long long)p.slot_mapping[row] : p.start_slot + row;
      if (slot < 0 || slot >= p.n_blocks * PAGE) { atomicOr(p.status, StatusBits::BAD_INDEX); continue; }
      const unsigned long long mask = p.row_masks ? p.row_masks[row] : p.agent_mask;
      float4 x0[8], x1[8];
#pragma unroll
      for (uint32_t s = 0; s < 8; ++s) {
        if (s < CS) {
          const float* src = recv + ((size_t)(s * (MT * 16) + row) * cpb + pc * 8);
          x0[s] = *reinterpret_cast<const float4*>(src);
          x1[s] = *reinterpret_cast<const float4*>(src + 4);
        } else {
          x0[s] = make_float4(0.f, 0.f, 0.f, 0.f); x1[s] = x0[s];
        }
      }
      float v8[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v8[k] = 0.f;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        v8[0] += x0[s].x; v8[1] += x0[s].y; v8[2] += x0[s].z; v8[3] += x0[s].w;
        v8[4] += x1[s].x; v8[5] += x1[s].y; v8[6] += x1[s].z; v8[7] += x1[s].w;
      }
      store_piece(p, slot / PAGE, (int)(slot % PAGE), gc, v8, mask, row);
    }
    return;     // a block leaves once everything addressed to it has arrived; its own sends carry their data with them
  }
  __syncthreads();                                     // all reads of the tiles are done; the region is reused

  // ---- partial tile [MT*16][COLS] fp32 -> shared memory
  float* part = reinterpret_cast<float*>(smem);
  if (warp < PS_WARPS) {
    const int r = lane >> 2, q = lane & 3;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        const int col = (warp * NT + t) * 8 + 2 * q;
        *reinterpret_cast<float2*>(part + (mt * 16 + r) * COLS + col) = make_float2(acc[mt][t][0], acc[mt][t][1]);
        *reinterpret_cast<float2*>(part + (mt * 16 + r + 8) * COLS + col) = make_float2(acc[mt][t][2], acc[mt][t][3]);
      }
  }
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");

  // ---- this block finishes columns [rank*COLS/CS, (rank+1)*COLS/CS) of its group: 8-column pieces,
  //      all peers' values requested at once, added in rank order
  const int pieces_per_row = COLS / 8 / CS;             // CS in {1,2,4,8}
  const uint32_t part_u32 = smem_u32(part);
  // eight columns [col, col+8) of one row, summed over the cluster's partial tiles
  auto gather = [&](int row, int col, float (&v8)[8]) {
    float4 x0[8], x1[8];
#pragma unroll
    for (uint32_t s = 0; s < 8; ++s) {
      if (s < CS) {
        uint32_t remote;
        asm("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote) : "r"(part_u32 + (row * COLS + col) * 4), "r"(s));
        asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(x0[s].x), "=f"(x0[s].y), "=f"(x0[s].z), "=f"(x0[s].w) : "r"(remote));
        asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(x1[s].x), "=f"(x1[s].y), "=f"(x1[s].z), "=f"(x1[s].w) : "r"(remote + 16));
      } else {
        x0[s] = make_float4(0.f, 0.f, 0.f, 0.f); x1[s] = x0[s];
      }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) v8[k] = 0.f;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      v8[0] += x0[s].x; v8[1] += x0[s].y; v8[2] += x0[s].z; v8[3] += x0[s].w;
      v8[4] += x1[s].x; v8[5] += x1[s].y; v8[6] += x1[s].z; v8[7] += x1[s].w;
    }
  };
  const int kw = (p.rope && p.mode != 0) ? p.n_kv * p.hd : 0;   // width of the key columns that get rotated
  for (int it = threadIdx.x; it < p.M * pieces_per_row; it += PS_THREADS) {
    const int row = it / pieces_per_row, pc = it % pieces_per_row;
    const int col = (rank * pieces_per_row + pc) * 8;
    const int gc = group * COLS + col;
    if (gc >= p.N_out) continue;
    if (gc < kw && (gc % p.hd) >= p.hd / 2) continue;   // upper half of a rotated head: written with its lower partner
    long long slot = p.slot_mapping ? (long long)p.slot_mapping[row] : p.start_slot + row;
    if (slot < 0 || slot >= p.n_blocks * PAGE) { atomicOr(p.status, StatusBits::BAD_INDEX); continue; }
    const unsigned long long mask = p.row_masks ? p.row_masks[row] : p.agent_mask;
    float v8[8];
    gather(row, col, v8);
    if (gc < kw) {
      // rotary keys: columns (c, c + hd/2) of a head turn by the row's position; the block tile holds whole
      // heads (COLS % hd == 0), so the partner piece sits hd/2 columns further in the same tiles
      long long pos = p.positions ? (long long)p.positions[row] : p.start_pos + row;
      if (pos < 0 || pos >= p.max_pos) { atomicOr(p.status, StatusBits::BAD_INDEX); continue; }
      float h8[8];
      gather(row, col + p.hd / 2, h8);
      const float4* cs = p.rope + pos * (p.hd / 4) + (gc % p.hd) / 2;
      float lo[8], hi[8];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 t4 = __ldg(cs + k);                // (cos c, sin c, cos c+1, sin c+1)
        lo[2 * k] = v8[2 * k] * t4.x - h8[2 * k] * t4.y;
        lo[2 * k + 1] = v8[2 * k + 1] * t4.z - h8[2 * k + 1] * t4.w;
        hi[2 * k] = h8[2 * k] * t4.x + v8[2 * k] * t4.y;
        hi[2 * k + 1] = h8[2 * k + 1] * t4.z + v8[2 * k + 1] * t4.w;
      }
      store_piece(p, slot / PAGE, (int)(slot % PAGE), gc, lo, mask, row);
      store_piece(p, slot / PAGE, (int)(slot % PAGE), gc + p.hd / 2, hi, mask, row);
      continue;
    }
    store_piece(p, slot / PAGE, (int)(slot % PAGE), gc, v8, mask, row);
  }
  // nobody leaves while a peer may still read its partial tile
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}

}  // namespace precc
