// Shared pieces of the tcgen05 / TMEM / TMA kernels: the projection parameters and tile constants, the sleeping
// form of the bounded mbarrier wait, TMA loads, shared-memory matrix descriptors, tcgen05.mma / commit / ld wrappers.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace precc {

struct GemmParams {
  int M, N_out, K;
  int BN, stages, tmem_cols;
  int spread_rows;                // 1: even row-tile spreading allowed (rows may be written twice, identically)
  int direct_send;                // split-K merge by sends: 1 = pieces straight from registers (st.async), 0 = whole slices by bulk copy
  int mode;                       // 0 = LR caches, 1 = base caches, 2 = base columns then LR columns
  const int32_t* slot_mapping;    // [M] or null
  int64_t start_slot;
  int64_t n_blocks;
  __nv_bfloat16* base_k;          // modes 1, 2
  __nv_bfloat16* base_v;
  __nv_bfloat16* lr_k;            // modes 0, 2
  __nv_bfloat16* lr_v;
  int n_agents, rank_k, rank_v;
  unsigned long long agent_mask;
  const unsigned long long* row_masks;   // optional [M]: per-row agent masks (double batching), overrides agent_mask
  const int32_t* lr_copy_slots;          // optional [M]: a second slot that also receives the row's LR rows (< 0: none)
  int n_kv, hd;
  int hd_shift, rk_shift, rv_shift;      // log2 of hd, rank_k, rank_v (all powers of two; 0 for an absent rank)
  // rotary keys (modes 1, 2; null = none): the key columns of a row are rotated by the row's position
  // before they are stored (rotate-half pairing (c, c + hd/2)); needs BN % hd == 0
  const float4* rope;             // [max_pos][hd/4] of (cos c, sin c, cos c+1, sin c+1), c even
  const int32_t* positions;       // [M] or null (start_pos + row)
  int64_t start_pos;
  int max_pos;
  uint32_t* status;
  unsigned long long* trace;      // PRECC_GEMM_TRACE builds only: [k-blocks][8] clock stamps of block 0
};

// Timeline stamps of the persistent GEMM's block 0 for tuning (compiled in with -DPRECC_GEMM_TRACE): slot 0 the
// producer sees the stage free, 1 its copies are issued, 2 the MMA lane sees the stage full, 3 its MMAs are issued,
// 4 the commit is issued.
#ifdef PRECC_GEMM_TRACE
#define GEMM_STAMP(p, it, slot)                                                                   \
  do {                                                                                            \
    if ((p).trace && blockIdx.x == 0 && (it) < 256) (p).trace[(it) * 8 + (slot)] = clock64();     \
  } while (0)
#else
#define GEMM_STAMP(p, it, slot) do { } while (0)
#endif

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;                 // 64 bf16 = one 128-byte swizzle row
constexpr int GEMM_THREADS = 192;
constexpr int GEMM_MAX_KS = 8;            // largest K split of the split-K kernels (cluster size)
constexpr int GEMM_PUSH_MAX_KS = 4;       // up to this split the partial tiles are merged by bulk sends
constexpr int GEMM_A_BYTES = GEMM_BM * GEMM_BK * 2;

// The same bounded wait for waiters that are not on the critical path (an epilogue waiting for a whole tile of
// MMAs): it sleeps between polls, so that four warps of waiters do not compete with the issuing lanes for issue
// slots - and for the power budget - while the tile is being computed.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  long long limit = -1;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      __nanosleep(200);
      if (mbar_try_wait(bar, parity)) return true;
    }
    if (limit < 0) limit = static_cast<long long>(*reinterpret_cast<volatile uint32_t*>(status + 1)) << 10;
    if (clock64() - t0 > limit) break;
    if (*reinterpret_cast<volatile uint32_t*>(status) & StatusBits::TIMEOUT) return false;
  }
  atomicOr(status, StatusBits::TIMEOUT);
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart (start >> 4 | LBO(ignored) | SBO = 1024 >> 4 | version 1 | layout SWIZZLE_128B).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFF) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// Instruction descriptor: D fp32, A/B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(GEMM_BM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}

}  // namespace precc
