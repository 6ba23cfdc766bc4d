// Device helpers shared by the precc kernels (sm_100a): async copies, ldmatrix, mma.sync
// fragments, bf16 packing and the swizzled shared-memory tile addressing.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace precc {

constexpr int PAGE = 16;
constexpr float NEG_BIG = -1.0e30f;   // finite stand-in for -inf in running maxima

struct StatusBits {
  static constexpr uint32_t BAD_INDEX = 1u;
  static constexpr uint32_t TIMEOUT = 2u;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte global -> shared copy that bypasses L1; src_bytes == 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];\n" : "=r"(r0), "=r"(r1) : "r"(addr));
}
// Transpose an 8x8 matrix of 16-bit elements held one row-pair per lane across the warp.
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// Programmatic dependent launch: when a kernel is launched with the programmatic-serialization
// attribute it may start while its predecessor in the stream drains; pdl_wait() blocks until the
// predecessor has completed and its writes are visible (a no-op for ordinary launches), and
// pdl_launch_dependents() lets the successor begin its own launch early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// ---- mbarrier basics (shared-memory address of the barrier as a 32-bit value)
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  `status` points at the context's two device words: [0] the status bits, [1] the wait limit in
// units of 1024 SM clock cycles (default: about a second).  Returns false after recording a timeout.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  long long limit = -1;                // fetched from global memory only once a whole batch of polls has failed:
  for (;;) {                           // the common short wait must not pay a memory round trip before it polls
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (limit < 0) limit = static_cast<long long>(*reinterpret_cast<volatile uint32_t*>(status + 1)) << 10;
    if (clock64() - t0 > limit) break;
    // once any wait in the grid has expired the results are void anyway: do not queue up more seconds
    if (*reinterpret_cast<volatile uint32_t*>(status) & StatusBits::TIMEOUT) return false;
  }
  atomicOr(status, StatusBits::TIMEOUT);
  return false;
}

// Bounded wait for bytes sent by other blocks of the cluster (acquire at cluster scope); limit as in mbar_wait.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, uint32_t* status) {
  auto poll = [&]() -> bool {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
  };
  if (poll()) return true;
  const long long t0 = clock64();
  long long limit = -1;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (poll()) return true;
    if (limit < 0) limit = static_cast<long long>(*reinterpret_cast<volatile uint32_t*>(status + 1)) << 10;
    if (clock64() - t0 > limit) break;
    if (*reinterpret_cast<volatile uint32_t*>(status) & StatusBits::TIMEOUT) return false;
  }
  atomicOr(status, StatusBits::TIMEOUT);
  return false;
}

// ---- distributed shared memory: address of a peer's copy of a shared-memory location, and stores that count
//      their bytes on an mbarrier of the receiving block
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_async_f32(uint32_t remote, float v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];\n"
               ::"r"(remote), "f"(v), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void st_async_b32x4(uint32_t remote, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];\n"
               ::"r"(remote), "r"(a), "r"(b), "r"(c), "r"(d), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void st_async_f32x2(uint32_t remote, float a, float b, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];\n"
               ::"r"(remote), "f"(a), "f"(b), "r"(remote_bar) : "memory");
}
// XOR swizzle of 16-byte chunks inside a tile whose rows hold CPR chunks (CPR in {1,2,4,8,16}):
// eight consecutive rows of the same logical chunk land in eight different 16-byte bank groups.
template <int CPR>
__device__ __forceinline__ int swz_chunk(int row, int chunk) {
  if constexpr (CPR >= 8) return chunk ^ (row & 7);
  else if constexpr (CPR == 4) return chunk ^ ((row >> 1) & 3);
  else if constexpr (CPR == 2) return chunk ^ ((row >> 2) & 1);
  else return chunk;
}
// Byte offset of (row, 16-byte chunk) in such a tile.
template <int CPR>
__device__ __forceinline__ int swz_off(int row, int chunk) {
  return (row * CPR + swz_chunk<CPR>(row, chunk)) * 16;
}

}  // namespace precc
