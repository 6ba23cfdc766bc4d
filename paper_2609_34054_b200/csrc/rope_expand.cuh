// Adapted rotary keys of one sequence, written out once for a turn's prefill (Appendix D.2: the key-side adapter
// term sits inside the rotation, so it cannot be folded into the query).  For every token t of the sequence,
// kv head g and column pair (c, c + hd/2):
//     K_a[t][g][:] = K_base_rot[t][g][:] + s_k RoPE_t( L^K_a[t][:] B^K_a[:, g] )
// with K_base_rot the cache's (already rotated) base keys, L^K the agent's unrotated LR rows and token t at
// position t.  The result goes to a caller-provided scratch area in LOGICAL block order, layout
// [block][kv head][16][hd] like the cache, so that the tensor-memory prefill kernel can stream it as its key
// operand with whole-stage boxes and no key-side adapter at all.  One thread block per 16-token block; a thread
// owns two adjacent columns of the lower half of a head and their partners in the upper half.
#pragma once
#include "common.cuh"

namespace precc {

struct RopeExpandParams {
  const __nv_bfloat16* k_base;   // [n_blocks][n_kv][16][hd]
  const __nv_bfloat16* lr_k;     // the agent's rows: [n_blocks][16][rk]
  const __nv_bfloat16* B_k;      // the agent's matrix: [rk][n_kv * hd]
  const float4* rope;            // [max_pos][hd/4] of (cos c, sin c, cos c+1, sin c+1), c even
  const int32_t* block_table;    // logical -> physical block, or null
  __nv_bfloat16* scratch;        // [n_out_blocks][n_kv][16][hd]
  uint32_t* status;
  long long n_blocks;            // physical blocks of the cache
  int first_block;               // physical block of logical block 0 when block_table is null
  int n_tokens;                  // tokens of the sequence (context + turn); rows past it are written as zeros
  int n_kv, hd, rk, max_pos;
  float s_k;
};

constexpr int RX_THREADS = 256;

__global__ void __launch_bounds__(RX_THREADS)
rope_expand_keys_kernel(const RopeExpandParams p) {
  __shared__ __align__(16) float Lf[64 * PAGE];          // s_k L^K of the block's tokens, [rank][token]
  const int lb = blockIdx.x;
  const int hd = p.hd, rk = p.rk;
  const int kvw = p.n_kv * hd;
  __nv_bfloat16* dst_blk = p.scratch + (size_t)lb * p.n_kv * PAGE * hd;
  const int t0 = lb * PAGE;
  if (t0 >= p.n_tokens) {                                // padding up to a whole 128-token stage: defined contents
    for (int i = threadIdx.x; i < p.n_kv * PAGE * hd / 8; i += RX_THREADS) reinterpret_cast<uint4*>(dst_blk)[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  int ph = p.block_table ? __ldg(p.block_table + lb) : p.first_block + lb;
  if (ph < 0 || ph >= p.n_blocks) {
    if (threadIdx.x == 0) atomicOr(p.status, StatusBits::BAD_INDEX);
    ph = 0;
  }
  for (int i = threadIdx.x; i < PAGE * rk; i += RX_THREADS) {
    const int tok = i / rk, j = i - tok * rk;
    Lf[j * PAGE + tok] = p.s_k * __bfloat162float(p.lr_k[((size_t)ph * PAGE + tok) * rk + j]);
  }
  __syncthreads();
  const int units = p.n_kv * (hd / 4);
  for (int u = threadIdx.x; u < units; u += RX_THREADS) {
    const int g = u / (hd / 4), cp = u - g * (hd / 4), c = 2 * cp;
    const __nv_bfloat16* bcol = p.B_k + (size_t)g * hd + c;
    const __nv_bfloat16* ksrc = p.k_base + ((size_t)ph * p.n_kv + g) * PAGE * hd + c;
    __nv_bfloat16* kdst = dst_blk + (size_t)g * PAGE * hd + c;
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
      float lo0[8], lo1[8], hi0[8], hi1[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) { lo0[t] = lo1[t] = hi0[t] = hi1[t] = 0.f; }
      for (int j = 0; j < rk; ++j) {
        const float2 bl = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(bcol + (size_t)j * kvw));
        const float2 bh = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(bcol + (size_t)j * kvw + hd / 2));
        const float4 la = *reinterpret_cast<const float4*>(Lf + j * PAGE + half * 8);
        const float4 lb4 = *reinterpret_cast<const float4*>(Lf + j * PAGE + half * 8 + 4);
        const float l8[8] = {la.x, la.y, la.z, la.w, lb4.x, lb4.y, lb4.z, lb4.w};
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          lo0[t] += l8[t] * bl.x; lo1[t] += l8[t] * bl.y;
          hi0[t] += l8[t] * bh.x; hi1[t] += l8[t] * bh.y;
        }
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int tok = half * 8 + t, pos = t0 + tok;
        __nv_bfloat162 olo = __floats2bfloat162_rn(0.f, 0.f), ohi = olo;
        if (pos < p.n_tokens) {
          const float4 cs = __ldg(p.rope + (size_t)min(pos, p.max_pos - 1) * (hd / 4) + cp);
          const float2 kl = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(ksrc + (size_t)tok * hd));
          const float2 kh = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(ksrc + (size_t)tok * hd + hd / 2));
          olo = __floats2bfloat162_rn(kl.x + (lo0[t] * cs.x - hi0[t] * cs.y), kl.y + (lo1[t] * cs.z - hi1[t] * cs.w));
          ohi = __floats2bfloat162_rn(kh.x + (hi0[t] * cs.x + lo0[t] * cs.y), kh.y + (hi1[t] * cs.z + lo1[t] * cs.w));
        }
        *reinterpret_cast<__nv_bfloat162*>(kdst + (size_t)tok * hd) = olo;
        *reinterpret_cast<__nv_bfloat162*>(kdst + (size_t)tok * hd + hd / 2) = ohi;
      }
    }
  }
}

}  // namespace precc
