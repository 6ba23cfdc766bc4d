// Adapted rotary keys of one sequence, written out once for a turn's prefill (Appendix D.2: the key-side adapter
// term sits inside the rotation, so it cannot be folded into the query).  For every token t of the sequence,
// kv head g and column pair (c, c + hd/2):
//     K_a[t][g][:] = K_base_rot[t][g][:] + s_k RoPE_t( L^K_a[t][:] B^K_a[:, g] )
// with K_base_rot the cache's (already rotated) base keys, L^K the agent's unrotated LR rows and token t at
// position t.  The result goes to a caller-provided scratch area in LOGICAL block order, layout
// [block][kv head][16][hd] like the cache, so that the tensor-memory prefill kernel can stream it as its key
// operand with whole-stage boxes and no key-side adapter at all.  One thread block per 16-token block.
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
  int n_out_blocks;              // cache blocks to write (whole 128-token stages)
  int n_kv, hd, rk, max_pos;
  float s_k;
};

constexpr int RX_THREADS = 256;
constexpr int RX_WARPS = RX_THREADS / 32;

// E = L^K B^K on the tensor cores (mma.sync m16n8k16: the 16 tokens of a cache block on the M axis, rank on K, columns
// on N).  A task is 16 adjacent columns of the lower half of one head together with their partners in the upper half;
// a warp owns TPW tasks for the whole kernel and keeps their B^K fragments in registers, a thread block owns a group
// of 8 TPW tasks (blockIdx.y) and walks over the sequence's cache blocks (blockIdx.x, persistent).  Per cache block:
// L^K fragments straight from global memory, the MMAs, the rotation, the scaled term parked in shared memory, then
// base keys + term -> scratch with 16-byte accesses, consecutive threads on consecutive pieces of a row.
// KS = k steps of 16 (rank 8 and 16: 1, rank 32: 2, rank 64: 4).
template <int KS>
struct RxCfg {
  static constexpr int GROUP_TASKS = RX_WARPS;           // one task per warp: 4 tiles * KS * 2 fragment registers
  static constexpr int PIECES = GROUP_TASKS * PAGE * 4 / RX_THREADS;   // 16-byte pieces of the group per thread and cache block
};

template <int KS>
__global__ void __launch_bounds__(RX_THREADS, 2)
rope_expand_keys_kernel(const RopeExpandParams p) {
  constexpr int PIECES = RxCfg<KS>::PIECES;
  extern __shared__ __align__(16) float Es[];            // s_k RoPE(L^K B^K) of one cache block, [task of the group][token][32 columns]
  const int hd = p.hd, rk = p.rk;
  const int kvw = p.n_kv * hd;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, q2 = (lane & 3) * 2;          // accumulator rows r, r + 8; columns q2, q2 + 1 of an 8-column tile
  const int tasks_per_head = hd / 32;                    // 16 lower-half columns per task
  const int n_tasks = p.n_kv * tasks_per_head;
  const int task = blockIdx.y * RxCfg<KS>::GROUP_TASKS + warp;
  const bool has_task = task < n_tasks;
  const int tg_head = task / tasks_per_head, tc0 = (task - tg_head * tasks_per_head) * 16;
  // ---- this warp's B^K fragments (k = rank, n = column), zero beyond the rank and beyond the last task
  uint32_t bfr[4][KS][2];
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int col = tg_head * hd + tc0 + (t & 1) * 8 + (t >> 1) * (hd / 2) + r;        // B operand: n = lane >> 2
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int k0 = ks * 16 + q2;
      auto bk = [&](int k) -> uint32_t {
        return (has_task && k < rk) ? (uint32_t)__bfloat16_as_ushort(p.B_k[(size_t)k * kvw + col]) : 0u;
      };
      bfr[t][ks][0] = bk(k0) | (bk(k0 + 1) << 16);
      bfr[t][ks][1] = bk(k0 + 8) | (bk(k0 + 9) << 16);
    }
  }
  // ---- the 16-byte pieces this thread combines per cache block: 8 columns of one token.  The group's tasks cover
  //      whole heads (8 tasks = 8 / tasks_per_head heads), and the pieces are taken in memory order - consecutive
  //      threads on consecutive pieces of a token's row of one head - so that every request covers whole 128-byte lines
  const int group_tasks = min(RxCfg<KS>::GROUP_TASKS, n_tasks - (int)blockIdx.y * RxCfg<KS>::GROUP_TASKS);
  const int ppr = hd / 8;                                  // pieces per row
  int p_off[PIECES], p_tok[PIECES], p_e[PIECES];
  bool p_on[PIECES];
#pragma unroll
  for (int k = 0; k < PIECES; ++k) {
    const int i = threadIdx.x + k * RX_THREADS;
    const int pr = i % ppr, tok = (i / ppr) % PAGE, hg = i / (ppr * PAGE);            // piece in row, token, head in group
    const int col = pr * 8, half = col >= hd / 2 ? 1 : 0, cl = col - half * (hd / 2);
    const int tg = hg * tasks_per_head + cl / 16;                                      // task in group that produced these columns
    const int g = blockIdx.y * (RxCfg<KS>::GROUP_TASKS / tasks_per_head) + hg;
    p_on[k] = tg < group_tasks;
    p_tok[k] = tok;
    p_off[k] = (g * PAGE + tok) * hd + col;
    p_e[k] = tg * PAGE * 32 + tok * 32 + half * 16 + (cl % 16);
  }
  // ---- inputs of one cache block, requested one block ahead of their use
  struct In {
    int ph;
    uint32_t afr[KS][4];        // L^K rows r and r + 8 (row-major [16][rk]); rank 8 fills half a k step
    float4 cs[2][2];            // (cos, sin) of the warp's columns at the lane's two tokens
    uint4 kb[PIECES];           // base keys of the thread's pieces
  };
  auto fetch = [&](int lb, In& x) {
    const int t0 = lb * PAGE;
    const bool pad = t0 >= p.n_tokens;
    int ph = 0;
    if (!pad) {
      ph = p.block_table ? __ldg(p.block_table + lb) : p.first_block + lb;
      if (ph < 0 || ph >= p.n_blocks) {
        if (threadIdx.x == 0 && blockIdx.y == 0) atomicOr(p.status, StatusBits::BAD_INDEX);
        ph = 0;
      }
    }
    x.ph = ph;
    const __nv_bfloat16* src_blk = p.k_base + (size_t)ph * p.n_kv * PAGE * hd;
#pragma unroll
    for (int k = 0; k < PIECES; ++k)
      x.kb[k] = (p_on[k] && t0 + p_tok[k] < p.n_tokens) ? __ldg(reinterpret_cast<const uint4*>(src_blk + p_off[k])) : make_uint4(0u, 0u, 0u, 0u);
    const __nv_bfloat16* lrow = p.lr_k + ((size_t)ph * PAGE + r) * rk;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int k = ks * 16 + q2;
      x.afr[ks][0] = (!pad && k < rk) ? __ldg(reinterpret_cast<const uint32_t*>(lrow + k)) : 0u;
      x.afr[ks][1] = (!pad && k < rk) ? __ldg(reinterpret_cast<const uint32_t*>(lrow + 8 * rk + k)) : 0u;
      x.afr[ks][2] = (!pad && k + 8 < rk) ? __ldg(reinterpret_cast<const uint32_t*>(lrow + k + 8)) : 0u;
      x.afr[ks][3] = (!pad && k + 8 < rk) ? __ldg(reinterpret_cast<const uint32_t*>(lrow + 8 * rk + k + 8)) : 0u;
    }
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int h = 0; h < 2; ++h)
        x.cs[t][h] = __ldg(p.rope + (size_t)min(t0 + r + 8 * h, p.max_pos - 1) * (hd / 4) + (tc0 + t * 8 + q2) / 2);
  };
  In cur;
  int lb = blockIdx.x;
  if (lb < p.n_out_blocks) fetch(lb, cur);
  for (; lb < p.n_out_blocks; lb += gridDim.x) {
    In nxt = cur;
    if (lb + (int)gridDim.x < p.n_out_blocks) fetch(lb + gridDim.x, nxt);           // in flight while this block is computed
    const int t0 = lb * PAGE;
    __nv_bfloat16* dst_blk = p.scratch + (size_t)lb * p.n_kv * PAGE * hd;
    if (has_task && t0 < p.n_tokens) {
      float acc[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) mma_bf16_16816(acc[t], cur.afr[ks], bfr[t][ks][0], bfr[t][ks][1]);
      }
      // rotate (lower tile t with upper tile t + 2), park the scaled term: [task in group][token][lower 16 | upper 16]
      float* eb = Es + (size_t)warp * PAGE * 32;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int cl = t * 8 + q2;                        // even column inside the task's lower 16
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int tok = r + 8 * h;
          const float lo0 = p.s_k * acc[t][2 * h], lo1 = p.s_k * acc[t][2 * h + 1];
          const float hi0 = p.s_k * acc[t + 2][2 * h], hi1 = p.s_k * acc[t + 2][2 * h + 1];
          const float4 cs = cur.cs[t][h];
          *reinterpret_cast<float2*>(eb + tok * 32 + cl) = make_float2(lo0 * cs.x - hi0 * cs.y, lo1 * cs.z - hi1 * cs.w);
          *reinterpret_cast<float2*>(eb + tok * 32 + 16 + cl) = make_float2(hi0 * cs.x + lo0 * cs.y, hi1 * cs.z + lo1 * cs.w);
        }
      }
    }
    __syncthreads();
    // base keys + term -> scratch (zeros past the sequence's end and in the padding up to a whole 128-token stage)
#pragma unroll
    for (int k = 0; k < PIECES; ++k) {
      if (!p_on[k]) continue;
      uint4 o = make_uint4(0u, 0u, 0u, 0u);
      if (t0 + p_tok[k] < p.n_tokens) {
        const float* e = Es + p_e[k];
        const float4 e0 = *reinterpret_cast<const float4*>(e), e1 = *reinterpret_cast<const float4*>(e + 4);
        auto add2 = [](uint32_t k2, float a, float b) -> uint32_t {
          const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&k2));
          return pack_bf16(f.x + a, f.y + b);
        };
        const uint4 kb = cur.kb[k];
        o = make_uint4(add2(kb.x, e0.x, e0.y), add2(kb.y, e0.z, e0.w), add2(kb.z, e1.x, e1.y), add2(kb.w, e1.z, e1.w));
      }
      *reinterpret_cast<uint4*>(dst_blk + p_off[k]) = o;
    }
    __syncthreads();                                     // the parked term is reused by the next cache block
    cur = nxt;
  }
}

template <int KS>
inline size_t rope_expand_smem_bytes() { return (size_t)RxCfg<KS>::GROUP_TASKS * PAGE * 32 * sizeof(float); }

}  // namespace precc
