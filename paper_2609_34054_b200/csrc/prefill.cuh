// LR-reconstructed attention for the S new tokens of a turn (context fully visible, new tokens
// causal).  Same algebra as decode: r_k extra contraction coordinates on the key side
// (q~ = s_k q B^K^T against the LR-K rows) and r_v extra output coordinates on the value side
// (U = P L^V, out += s_v U B^V), so the agent's K and V are never formed.
//
// One thread block = 64 query rows of one kv head, a row being (new token i, head within the
// group): row = i*G + hg.  Four warps x 16 rows; 64-token tiles of {K, V, L^K, L^V} stream through
// a cp.async ring shared by the block; S = Q'K'^T and O' += P V' run on mma.sync m16n8k16 with the
// FlashAttention-2 register reuse of P.
//
// Rotary variant (ROPE = true, Appendix D.2: rotated base keys, un-rotated LR-K rows): before a tile
// is used, each warp expands E = L^K (s_k B^K_g) for 16 of the tile's tokens on the tensor cores, rotates
// it by the tokens' positions (cached token t sits at position t) and adds it onto the key rows in
// shared memory, so that the score MMA sees the agent's rotated keys; the fold q~ is not used.  The
// agent's keys exist only in that shared-memory tile.
#pragma once
#include "common.cuh"

namespace precc {

struct PrefillParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int32_t* block_table;
  const __nv_bfloat16* k_base;
  const __nv_bfloat16* v_base;
  const __nv_bfloat16* lr_k;   // already offset to the agent
  const __nv_bfloat16* lr_v;
  const __nv_bfloat16* B_k;    // already offset to the agent: [r][n_kv*hd]
  const __nv_bfloat16* B_v;
  uint32_t* status;
  int64_t n_blocks;
  int S, T, first_block;
  int n_q, n_kv, group;
  int stages;
  float scale_log2, s_k, s_v;
  const float4* rope;          // rotary variant: [max_pos][hd/4] of (cos c, sin c, cos c+1, sin c+1), c even
  int max_pos;
};

constexpr int PF_ROWS = 64;
constexpr int PF_TOK = 64;
constexpr int PF_THREADS = 128;

template <int HD, int RK, int RV>
struct PrefillCfg {
  static constexpr int RKP = RK == 0 ? 0 : (RK < 16 ? 16 : RK);
  static constexpr int Q_BYTES = PF_ROWS * HD * 2;
  static constexpr int QX_BYTES = PF_ROWS * RKP * 2;
  static constexpr int KV_BYTES = PF_TOK * HD * 2;
  static constexpr int LK_BYTES = PF_TOK * RK * 2;
  static constexpr int LV_BYTES = PF_TOK * RV * 2;
  static constexpr int STAGE_BYTES = 2 * KV_BYTES + LK_BYTES + LV_BYTES;
  static constexpr int OW = HD + RV;
  static constexpr int BK_BYTES = (RK > 16 ? RK : 16) * HD * 2;   // rotary variant: s_k B^K_g slice, rows padded to 16
  __host__ __device__ static constexpr int smem_bytes(int stages, bool rope = false) {
    int stream = Q_BYTES + QX_BYTES + stages * STAGE_BYTES + (rope ? BK_BYTES : 0);
    int epi = PF_ROWS * (OW + 1) * 4;
    return (stream > epi ? stream : epi) + 16;
  }
};

template <int HD, int RK, int RV, bool ROPE = false>
__global__ void __launch_bounds__(PF_THREADS)
lr_attend_prefill_kernel(const PrefillParams p) {
  static_assert(!ROPE || RK > 0, "the rotary variant only differs when there is a key-side adapter");
  using C = PrefillCfg<HD, RK, RV>;
  constexpr int OW = C::OW;
  constexpr int KC = HD / 16;
  constexpr int KX = C::RKP / 16;
  constexpr int NO = HD / 8;                  // output n-tiles (base)
  constexpr int NX = RV / 8;                  // output n-tiles (LR-V)
  constexpr int CPR_KV = HD / 8;
  constexpr int CPR_QX = C::RKP > 0 ? C::RKP / 8 : 1;
  constexpr int CPR_LK = RK > 0 ? RK / 8 : 1;
  constexpr int CPR_LV = RV > 0 ? RV / 8 : 1;

  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.y;
  const int G = p.group;
  // block x = 0 takes the LAST row tile: blocks with the longest causal reach start first, the grid's tail is short blocks
  const int row0 = (int)(gridDim.x - 1 - blockIdx.x) * PF_ROWS;      // first (token, head) row of this block
  const int n_rows = p.S * G;

  const uint32_t q_u32 = smem_u32(smem);
  const uint32_t qx_u32 = q_u32 + C::Q_BYTES;
  const uint32_t ring_u32 = qx_u32 + C::QX_BYTES;

  const int i_min = row0 / G;
  const int i_max = min(p.S - 1, (row0 + PF_ROWS - 1) / G);
  const int t_end = p.T + i_max + 1;          // tokens this block attends
  const int n_tiles = (t_end + PF_TOK - 1) / PF_TOK;
  const int full_vis = p.T + i_min + 1;       // tokens visible to every row of the block

  auto issue_tile = [&](int it) {
    if (it < n_tiles) {
      const uint32_t st = ring_u32 + (uint32_t)(it % p.stages) * C::STAGE_BYTES;
      // 4 pages of 16 tokens; thread block covers each page's K and V with 16-byte chunks
      for (int pg = 0; pg < PF_TOK / PAGE; ++pg) {
        const int lt = it * (PF_TOK / PAGE) + pg;              // logical block
        const bool live = lt * PAGE < t_end;
        int ph = 0;
        if (live) {
          ph = p.block_table ? p.block_table[lt] : p.first_block + lt;
          if (ph < 0 || ph >= p.n_blocks) { if (threadIdx.x == 0) atomicOr(p.status, StatusBits::BAD_INDEX); ph = 0; }
        }
        // rows past the last attended token are zero-filled: their weights are zero, but 0 * garbage
        // (an unwritten slot may hold NaN) must not reach the accumulators
        const int n_ok = live ? min(PAGE, t_end - lt * PAGE) : 0;
        const unsigned char* ksrc = reinterpret_cast<const unsigned char*>(p.k_base + ((size_t)ph * p.n_kv + g) * PAGE * HD);
        const unsigned char* vsrc = reinterpret_cast<const unsigned char*>(p.v_base + ((size_t)ph * p.n_kv + g) * PAGE * HD);
        for (int c = threadIdx.x; c < PAGE * CPR_KV; c += PF_THREADS) {
          const int row = pg * PAGE + c / CPR_KV, ch = c % CPR_KV;
          const int off = swz_off<CPR_KV>(row, ch);
          const int ok = (c / CPR_KV) < n_ok ? 16 : 0;
          cp_async16(st + off, ksrc + c * 16, ok);
          cp_async16(st + C::KV_BYTES + off, vsrc + c * 16, ok);
        }
        if constexpr (RK > 0) {
          const unsigned char* src = reinterpret_cast<const unsigned char*>(p.lr_k + (size_t)ph * PAGE * RK);
          for (int c = threadIdx.x; c < PAGE * CPR_LK; c += PF_THREADS) {
            const int row = pg * PAGE + c / CPR_LK, ch = c % CPR_LK;
            cp_async16(st + 2 * C::KV_BYTES + swz_off<CPR_LK>(row, ch), src + c * 16, (c / CPR_LK) < n_ok ? 16 : 0);
          }
        }
        if constexpr (RV > 0) {
          const unsigned char* src = reinterpret_cast<const unsigned char*>(p.lr_v + (size_t)ph * PAGE * RV);
          for (int c = threadIdx.x; c < PAGE * CPR_LV; c += PF_THREADS) {
            const int row = pg * PAGE + c / CPR_LV, ch = c % CPR_LV;
            cp_async16(st + 2 * C::KV_BYTES + C::LK_BYTES + swz_off<CPR_LV>(row, ch), src + c * 16, (c / CPR_LV) < n_ok ? 16 : 0);
          }
        }
      }
    }
    cp_async_commit();
  };
  for (int it = 0; it < p.stages - 1; ++it) issue_tile(it);

  // ---- Q tile (zero rows past the end) and the folded key-side adapter q~
  for (int c = threadIdx.x; c < PF_ROWS * CPR_KV; c += PF_THREADS) {
    const int r = c / CPR_KV, ch = c % CPR_KV;
    const int row = row0 + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < n_rows) {
      const int i = row / G, hg = row % G;
      v = *reinterpret_cast<const uint4*>(p.q + ((size_t)i * p.n_q + (size_t)g * G + hg) * HD + ch * 8);
    }
    *reinterpret_cast<uint4*>(smem + swz_off<CPR_KV>(r, ch)) = v;
  }
  const uint32_t bk_u32 = ring_u32 + p.stages * C::STAGE_BYTES;
  if constexpr (ROPE) {
    // s_k B^K[:, g] -> shared memory, [max(RK,16)][HD], swizzled like a key tile (rows >= RK are zero)
    constexpr int ROWS = RK > 16 ? RK : 16;
    for (int c = threadIdx.x; c < ROWS * CPR_KV; c += PF_THREADS) {
      const int j = c / CPR_KV, ch = c % CPR_KV;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (j < RK) v = __ldg(reinterpret_cast<const uint4*>(p.B_k + (size_t)j * p.n_kv * HD + (size_t)g * HD + ch * 8));
      auto sc = [&](uint32_t x) -> uint32_t {
        const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x));
        return pack_bf16(f.x * p.s_k, f.y * p.s_k);
      };
      *reinterpret_cast<uint4*>(smem + (bk_u32 - q_u32) + swz_off<CPR_KV>(j, ch)) = make_uint4(sc(v.x), sc(v.y), sc(v.z), sc(v.w));
    }
  }
  if constexpr (RK > 0 && !ROPE) {
    for (int e = threadIdx.x; e < PF_ROWS * C::RKP; e += PF_THREADS) {
      const int r = e / C::RKP, j = e % C::RKP;
      const int row = row0 + r;
      float acc = 0.f;
      if (row < n_rows && j < RK) {
        const int i = row / G, hg = row % G;
        const uint4* qv = reinterpret_cast<const uint4*>(p.q + ((size_t)i * p.n_q + (size_t)g * G + hg) * HD);
        const uint4* bv = reinterpret_cast<const uint4*>(p.B_k + (size_t)j * p.n_kv * HD + (size_t)g * HD);
#pragma unroll 4
        for (int c = 0; c < HD / 8; ++c) {
          uint4 x = __ldg(qv + c), y = __ldg(bv + c);
          const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            acc += bf16_bits_to_float(xs[k] & 0xffff) * bf16_bits_to_float(ys[k] & 0xffff);
            acc += bf16_bits_to_float(xs[k] >> 16) * bf16_bits_to_float(ys[k] >> 16);
          }
        }
      }
      __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(smem + C::Q_BYTES + swz_off<CPR_QX>(r, j / 8)) + (j % 8);
      *dst = __float2bfloat16(acc * p.s_k);
    }
  }

  float o[NO + NX][4];
#pragma unroll
  for (int i = 0; i < NO + NX; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_r[2] = {NEG_BIG, NEG_BIG}, l_r[2] = {0.f, 0.f};
  // causal limits of this lane's two rows (inclusive last visible token); rows past the end see nothing
  int lim[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = row0 + warp * 16 + (lane >> 2) + 8 * h;
    lim[h] = row < n_rows ? p.T + row / G : -1;
  }

  const int qa_row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;   // Q' A-operand
  const int qa_cpar = lane >> 4;
  const int kb_row = (lane & 7) + (lane >> 4) * 8;                      // K' B-operand (two n-tiles)
  const int kb_cpar = (lane >> 3) & 1;
  const int vb_row = (lane & 7) + ((lane >> 3) & 1) * 8;                // V' B-operand (transposed load)
  const int vb_cpar = lane >> 4;

  for (int it = 0; it < n_tiles; ++it) {
    switch (p.stages) {
      case 2: cp_async_wait<0>(); break;
      default: cp_async_wait<1>(); break;
    }
    __syncthreads();
    issue_tile(it + p.stages - 1);
    const uint32_t st = ring_u32 + (uint32_t)(it % p.stages) * C::STAGE_BYTES;
    const int t0 = it * PF_TOK;

    if constexpr (ROPE) {
      // this warp's 16 tokens of the tile: K[tok] += RoPE_tok(L^K[tok] . s_k B^K_g), in shared memory
      constexpr int KH = KC / 2;
      constexpr int KXR = (RK + 15) / 16;
      const int ar = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, ac = lane >> 4;   // A operand rows / chunk parity
      const int br = (lane & 7) + ((lane >> 3) & 1) * 8, bc = lane >> 4;                // B^K slice rows / chunk parity
      const int r0 = warp * 16 + (lane >> 2), qk = (lane & 3) * 2;
      uint32_t la[KXR][4];
#pragma unroll
      for (int jx = 0; jx < KXR; ++jx) {
        if constexpr (RK >= 16) {
          ldsm_x4(la[jx], st + 2 * C::KV_BYTES + swz_off<CPR_LK>(ar, 2 * jx + ac));
        } else {
          la[jx][2] = 0u; la[jx][3] = 0u;
          ldsm_x2(la[jx][0], la[jx][1], st + 2 * C::KV_BYTES + swz_off<1>(ar, 0));
        }
      }
      const int pos0 = min(t0 + r0, p.max_pos - 1), pos1 = min(t0 + r0 + 8, p.max_pos - 1);
#pragma unroll
      for (int kc = 0; kc < KH; ++kc) {
        float e[2][2][4];                               // [half][n-tile][c]
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
          for (int n2 = 0; n2 < 2; ++n2) { e[hf][n2][0] = e[hf][n2][1] = e[hf][n2][2] = e[hf][n2][3] = 0.f; }
#pragma unroll
          for (int jx = 0; jx < KXR; ++jx) {
            uint32_t bf[4];
            ldsm_x4_t(bf, bk_u32 + swz_off<CPR_KV>(16 * jx + br, 2 * (kc + hf * KH) + bc));
            mma_bf16_16816(e[hf][0], la[jx], bf[0], bf[1]);
            mma_bf16_16816(e[hf][1], la[jx], bf[2], bf[3]);
          }
        }
#pragma unroll
        for (int n2 = 0; n2 < 2; ++n2)
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const int col = kc * 16 + n2 * 8 + qk;                       // lower-half column (even)
            const float4 c4 = __ldg(p.rope + (size_t)(r ? pos1 : pos0) * (HD / 4) + (col >> 1));
            const float lo0 = e[0][n2][2 * r], lo1 = e[0][n2][2 * r + 1];
            const float hi0 = e[1][n2][2 * r], hi1 = e[1][n2][2 * r + 1];
            const uint32_t rl = pack_bf16(lo0 * c4.x - hi0 * c4.y, lo1 * c4.z - hi1 * c4.w);
            const uint32_t rh = pack_bf16(hi0 * c4.x + lo0 * c4.y, hi1 * c4.z + lo1 * c4.w);
            const int row = r0 + 8 * r;
            __nv_bfloat162* klo = reinterpret_cast<__nv_bfloat162*>(smem + (st - q_u32) + swz_off<CPR_KV>(row, col >> 3) + (col & 7) * 2);
            __nv_bfloat162* khi = reinterpret_cast<__nv_bfloat162*>(smem + (st - q_u32) + swz_off<CPR_KV>(row, (col + HD / 2) >> 3) + (col & 7) * 2);
            *klo = __hadd2(*klo, *reinterpret_cast<const __nv_bfloat162*>(&rl));
            *khi = __hadd2(*khi, *reinterpret_cast<const __nv_bfloat162*>(&rh));
          }
      }
      __syncthreads();                                   // every warp's 16 tokens are updated before any warp reads keys
    }

    float s[PF_TOK / 8][4];
#pragma unroll
    for (int nt = 0; nt < PF_TOK / 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
    for (int kc = 0; kc < KC; ++kc) {
      uint32_t a[4];
      ldsm_x4(a, q_u32 + swz_off<CPR_KV>(qa_row, 2 * kc + qa_cpar));
#pragma unroll
      for (int n2 = 0; n2 < PF_TOK / 16; ++n2) {
        uint32_t b[4];
        ldsm_x4(b, st + swz_off<CPR_KV>(n2 * 16 + kb_row, 2 * kc + kb_cpar));
        mma_bf16_16816(s[2 * n2], a, b[0], b[1]);
        mma_bf16_16816(s[2 * n2 + 1], a, b[2], b[3]);
      }
    }
    if constexpr (RK > 0 && !ROPE) {
#pragma unroll
      for (int kc = 0; kc < KX; ++kc) {
        uint32_t a[4];
        ldsm_x4(a, qx_u32 + swz_off<CPR_QX>(qa_row, 2 * kc + qa_cpar));
#pragma unroll
        for (int n2 = 0; n2 < PF_TOK / 16; ++n2) {
          if constexpr (RK >= 16) {
            uint32_t b[4];
            ldsm_x4(b, st + 2 * C::KV_BYTES + swz_off<CPR_LK>(n2 * 16 + kb_row, 2 * kc + kb_cpar));
            mma_bf16_16816(s[2 * n2], a, b[0], b[1]);
            mma_bf16_16816(s[2 * n2 + 1], a, b[2], b[3]);
          } else {
            uint32_t b0, b1;   // rank 8: one 16-byte chunk per token; upper half of the k-chunk is zero
            ldsm_x2(b0, b1, st + 2 * C::KV_BYTES + swz_off<1>(n2 * 16 + (lane & 15), 0));
            mma_bf16_16816(s[2 * n2], a, b0, 0u);
            mma_bf16_16816(s[2 * n2 + 1], a, b1, 0u);
          }
        }
      }
    }

    // ---- scale, mask, online softmax (rows lane>>2 and +8; columns 2*(lane&3), +1 of each n-tile)
    const bool need_mask = t0 + PF_TOK > full_vis || lim[0] < 0 || lim[1] < 0;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < PF_TOK / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float z = s[nt][e] * p.scale_log2;
        if (need_mask) {
          const int t = t0 + nt * 8 + (lane & 3) * 2 + (e & 1);
          if (t > lim[e >> 1]) z = -INFINITY;
        }
        s[nt][e] = z;
        mx[e >> 1] = fmaxf(mx[e >> 1], z);
      }
    }
    float al[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float mn = fmaxf(m_r[h], mx[h]);
      al[h] = fast_exp2(m_r[h] - mn);
      m_r[h] = mn;
      l_r[h] *= al[h];
    }
#pragma unroll
    for (int nt = 0; nt < PF_TOK / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float pv = fast_exp2(s[nt][e] - m_r[e >> 1]);
        s[nt][e] = pv;
        l_r[e >> 1] += pv;
      }
    }
#pragma unroll
    for (int i = 0; i < NO + NX; ++i) { o[i][0] *= al[0]; o[i][1] *= al[0]; o[i][2] *= al[1]; o[i][3] *= al[1]; }

    // ---- O' += P V'
#pragma unroll
    for (int j = 0; j < PF_TOK / 16; ++j) {
      uint32_t a[4];
      a[0] = pack_bf16(s[2 * j][0], s[2 * j][1]);
      a[1] = pack_bf16(s[2 * j][2], s[2 * j][3]);
      a[2] = pack_bf16(s[2 * j + 1][0], s[2 * j + 1][1]);
      a[3] = pack_bf16(s[2 * j + 1][2], s[2 * j + 1][3]);
#pragma unroll
      for (int np = 0; np < NO / 2; ++np) {
        uint32_t b[4];
        ldsm_x4_t(b, st + C::KV_BYTES + swz_off<CPR_KV>(j * 16 + vb_row, 2 * np + vb_cpar));
        mma_bf16_16816(o[2 * np], a, b[0], b[1]);
        mma_bf16_16816(o[2 * np + 1], a, b[2], b[3]);
      }
      if constexpr (RV >= 16) {
#pragma unroll
        for (int np = 0; np < NX / 2; ++np) {
          uint32_t b[4];
          ldsm_x4_t(b, st + 2 * C::KV_BYTES + C::LK_BYTES + swz_off<CPR_LV>(j * 16 + vb_row, 2 * np + vb_cpar));
          mma_bf16_16816(o[NO + 2 * np], a, b[0], b[1]);
          mma_bf16_16816(o[NO + 2 * np + 1], a, b[2], b[3]);
        }
      } else if constexpr (RV == 8) {
        uint32_t b0, b1;
        ldsm_x2_t(b0, b1, st + 2 * C::KV_BYTES + C::LK_BYTES + swz_off<1>(j * 16 + (lane & 15), 0));
        mma_bf16_16816(o[NO], a, b0, b1);
      }
    }
  }
  cp_async_wait<0>();
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_r[h] += __shfl_xor_sync(0xffffffffu, l_r[h], 1);
    l_r[h] += __shfl_xor_sync(0xffffffffu, l_r[h], 2);
  }
  __syncthreads();     // the ring is no longer read: reuse shared memory for the epilogue tile

  // ---- epilogue tile: eo[row][OW] (fp32) and el[row]
  float* eo = reinterpret_cast<float*>(smem);
  float* el = eo + PF_ROWS * OW;
  {
    const int r = warp * 16 + (lane >> 2), cq = (lane & 3) * 2;
#pragma unroll
    for (int i = 0; i < NO + NX; ++i) {
      eo[r * OW + i * 8 + cq] = o[i][0];
      eo[r * OW + i * 8 + cq + 1] = o[i][1];
      eo[(r + 8) * OW + i * 8 + cq] = o[i][2];
      eo[(r + 8) * OW + i * 8 + cq + 1] = o[i][3];
    }
    if ((lane & 3) == 0) { el[r] = l_r[0]; el[r + 8] = l_r[1]; }
  }
  __syncthreads();
  // out[row][c] = (O[row][c] + s_v * sum_j U[row][j] * B_v[j][g*hd + c]) / l[row]
  for (int e = threadIdx.x; e < PF_ROWS * (HD / 2); e += PF_THREADS) {
    const int r = e / (HD / 2), c = (e % (HD / 2)) * 2;
    const int row = row0 + r;
    if (row >= n_rows) continue;
    float v0 = eo[r * OW + c], v1 = eo[r * OW + c + 1];
    if constexpr (RV > 0) {
      float u0 = 0.f, u1 = 0.f;
#pragma unroll 8
      for (int j = 0; j < RV; ++j) {
        const float u = eo[r * OW + HD + j];
        const __nv_bfloat162 bb = *reinterpret_cast<const __nv_bfloat162*>(p.B_v + (size_t)j * p.n_kv * HD + (size_t)g * HD + c);
        u0 += u * __low2float(bb);
        u1 += u * __high2float(bb);
      }
      v0 += p.s_v * u0;
      v1 += p.s_v * u1;
    }
    const float inv = 1.f / el[r];
    const int i = row / G, hg = row % G;
    *reinterpret_cast<__nv_bfloat162*>(p.out + ((size_t)i * p.n_q + (size_t)g * G + hg) * HD + c) =
        __floats2bfloat162_rn(v0 * inv, v1 * inv);
  }
}

}  // namespace precc
