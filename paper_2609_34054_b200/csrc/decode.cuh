// LR-reconstructed decode attention (split-KV).
//
// For request b (agent a), kv head g and its G <= 8 query heads the kernel evaluates plain softmax
// attention with K_a = K_base + s_k L^K_a B^K_a and V_a = V_base + s_v L^V_a B^V_a (Eq. 1) without
// building K_a or V_a: the key-side adapter is folded into r extra query coordinates
// (q~ = s_k q B^K_{a,g}^T, contraction length head_dim + r_k) and the value-side adapter into r extra
// output coordinates (U = P L^V_a, then out += s_v U B^V_{a,g}).
//
// Work split: grid (split j, kv head g, request b).  A thread block owns `chunk_tiles` consecutive
// 16-token pages of one (b, g); its warps take pages round-robin, each with a private cp.async ring
// (no block-wide barrier inside the stream loop).  Tokens sit on the MMA M axis:
//   S^T[16 tok x 8 q]   = K'[16 x (hd+r_k)] . Q'^T          (mma.sync m16n8k16, bf16 -> fp32)
//   O^T[(hd+r_v) x 8 q] += V'^T[(hd+r_v) x 16 tok] . P^T     (P^T obtained with movmatrix)
// so no MMA row is wasted on padding.  Per-block partial (m, l, O') goes to the workspace; the last
// block to finish a (b, g) (atomic ticket) merges the partials in split order and applies the
// B^V epilogue.  Nothing waits on another block.
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
  float* part;        // [B][n_kv][max_splits][PART_STRIDE]
  int32_t* tickets;   // [B][n_kv], zero between calls
  uint32_t* status;
  int64_t n_blocks;
  int table_stride;
  int n_q, n_kv, group, n_agents;
  int chunk_tiles, max_splits, stages;
  float scale_log2, s_k, s_v;
};

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;

template <int HD, int RK, int RV>
struct DecodeCfg {
  static constexpr int KV_BYTES = PAGE * HD * 2;
  static constexpr int LK_BYTES = PAGE * RK * 2;
  static constexpr int LV_BYTES = PAGE * RV * 2;
  static constexpr int STAGE_BYTES = 2 * KV_BYTES + LK_BYTES + LV_BYTES;
  static constexpr int OW = HD + RV;                 // accumulated output width
  static constexpr int PART_STRIDE = 8 * OW + 16;     // floats: m[8], l[8], O'[8][OW]
  static constexpr int QX_BYTES = 8 * (RK > 0 ? RK : 8) * 2;
  static constexpr int MERGE_FLOATS = DEC_WARPS * (OW * 8 + 16);
  static constexpr int smem_bytes(int stages) {
    int ring = DEC_WARPS * stages * STAGE_BYTES;
    int merge = MERGE_FLOATS * 4;
    return (ring > merge ? ring : merge) + QX_BYTES + 64;
  }
};

template <int HD, int RK, int RV>
__global__ void __launch_bounds__(DEC_THREADS)
lr_attend_decode_kernel(const DecodeParams p) {
  using C = DecodeCfg<HD, RK, RV>;
  constexpr int OW = C::OW;
  constexpr int KC = HD / 16;                         // k-chunks of the base part
  constexpr int KX = (RK + 15) / 16;                  // k-chunks of the LR-K part
  constexpr int MT = HD / 16;                         // m-tiles of the base output
  constexpr int MX = (RV + 15) / 16;                  // m-tiles of the LR-V output
  constexpr int CPR_KV = HD / 8;
  constexpr int CPR_LK = RK > 0 ? RK / 8 : 1;
  constexpr int CPR_LV = RV > 0 ? RV / 8 : 1;

  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int G = p.group;

  const int ctx = p.ctx_len[b];
  const int agent = p.agent_id[b];
  __nv_bfloat16* out_bg = p.out + ((size_t)b * p.n_q + (size_t)g * G) * HD;
  if (ctx < 1 || agent < 0 || agent >= p.n_agents) {
    if (split == 0) {
      for (int i = threadIdx.x; i < G * HD; i += DEC_THREADS) out_bg[i] = __float2bfloat16(0.f);
      if (threadIdx.x == 0 && ctx >= 1) atomicOr(p.status, StatusBits::BAD_INDEX);
    }
    return;
  }
  const int n_tiles = (ctx + PAGE - 1) / PAGE;
  const int n_splits = (n_tiles + p.chunk_tiles - 1) / p.chunk_tiles;
  if (split >= n_splits) return;
  const int tile0 = split * p.chunk_tiles;
  const int tile_end = min(n_tiles, tile0 + p.chunk_tiles);
  // this warp's tiles: tile0 + warp + DEC_WARPS * i
  const int my_n = (tile_end - tile0 - warp + DEC_WARPS - 1) / DEC_WARPS;   // may be <= 0

  unsigned char* ring = smem + (size_t)warp * p.stages * C::STAGE_BYTES;
  const uint32_t ring_u32 = smem_u32(ring);
  const int ring_total = DEC_WARPS * p.stages * C::STAGE_BYTES;
  const int merge_total = C::MERGE_FLOATS * 4;
  __nv_bfloat16* qx = reinterpret_cast<__nv_bfloat16*>(smem + (ring_total > merge_total ? ring_total : merge_total));

  // ---- physical block ids, fetched 32 tiles at a time, one batch ahead
  auto load_phys = [&](int batch) -> int {
    int i = batch * 32 + lane;
    int t = tile0 + warp + DEC_WARPS * i;
    if (i >= my_n) return 0;
    int ph = p.block_table ? p.block_table[(size_t)b * p.table_stride + t]
                           : (p.first_block ? p.first_block[b] : 0) + t;
    if (ph < 0 || ph >= p.n_blocks) { atomicOr(p.status, StatusBits::BAD_INDEX); ph = 0; }
    return ph;
  };
  int phys_cur = load_phys(0);
  int phys_nxt = load_phys(1);

  const __nv_bfloat16* lrk_a = RK > 0 ? p.lr_k + (size_t)agent * p.n_blocks * PAGE * RK : nullptr;
  const __nv_bfloat16* lrv_a = RV > 0 ? p.lr_v + (size_t)agent * p.n_blocks * PAGE * RV : nullptr;

  auto issue_tile = [&](int i) {
    if (i < my_n) {
      if ((i & 31) == 0 && i > 0) { phys_cur = phys_nxt; phys_nxt = load_phys((i >> 5) + 1); }
      const int ph = __shfl_sync(0xffffffffu, phys_cur, i & 31);
      const int t = tile0 + warp + DEC_WARPS * i;
      const int valid = min(PAGE, ctx - t * PAGE);
      const uint32_t st = ring_u32 + (uint32_t)(i % p.stages) * C::STAGE_BYTES;
      const unsigned char* ksrc = reinterpret_cast<const unsigned char*>(p.k_base + ((size_t)ph * p.n_kv + g) * PAGE * HD);
      const unsigned char* vsrc = reinterpret_cast<const unsigned char*>(p.v_base + ((size_t)ph * p.n_kv + g) * PAGE * HD);
#pragma unroll
      for (int c = lane; c < PAGE * CPR_KV; c += 32) {
        const int row = c / CPR_KV, ch = c % CPR_KV;
        const int off = swz_off<CPR_KV>(row, ch);
        cp_async16(st + off, ksrc + c * 16, 16);
        cp_async16(st + C::KV_BYTES + off, vsrc + c * 16, row < valid ? 16 : 0);
      }
      if constexpr (RK > 0) {
        const unsigned char* src = reinterpret_cast<const unsigned char*>(lrk_a + (size_t)ph * PAGE * RK);
#pragma unroll
        for (int c = lane; c < PAGE * CPR_LK; c += 32) {
          const int row = c / CPR_LK, ch = c % CPR_LK;
          cp_async16(st + 2 * C::KV_BYTES + swz_off<CPR_LK>(row, ch), src + c * 16, 16);
        }
      }
      if constexpr (RV > 0) {
        const unsigned char* src = reinterpret_cast<const unsigned char*>(lrv_a + (size_t)ph * PAGE * RV);
#pragma unroll
        for (int c = lane; c < PAGE * CPR_LV; c += 32) {
          const int row = c / CPR_LV, ch = c % CPR_LV;
          cp_async16(st + 2 * C::KV_BYTES + C::LK_BYTES + swz_off<CPR_LV>(row, ch), src + c * 16, row < valid ? 16 : 0);
        }
      }
    }
    cp_async_commit();
  };

  // ---- start the stream before anything else
  for (int i = 0; i < p.stages - 1; ++i) issue_tile(i);

  // ---- query fragments: B operand (k = head-dim coordinate, n = query head)
  const int qrow = lane >> 2;                 // query head within the group held as column n
  const int qk = (lane & 3) * 2;
  uint32_t qb[KC][2];
  {
    const __nv_bfloat16* qsrc = p.q + ((size_t)b * p.n_q + (size_t)g * G + qrow) * HD;
#pragma unroll
    for (int kc = 0; kc < KC; ++kc) {
      if (qrow < G) {
        qb[kc][0] = *reinterpret_cast<const uint32_t*>(qsrc + kc * 16 + qk);
        qb[kc][1] = *reinterpret_cast<const uint32_t*>(qsrc + kc * 16 + 8 + qk);
      } else {
        qb[kc][0] = 0u; qb[kc][1] = 0u;
      }
    }
  }
  // ---- folded key-side adapter: q~[h][j] = s_k * sum_c q[h][c] * B_k[a][j][g*hd + c]
  uint32_t qxb[KX > 0 ? KX : 1][2];
  if constexpr (RK > 0) {
    const __nv_bfloat16* Bk = p.B_k + ((size_t)agent * RK) * ((size_t)p.n_kv * HD) + (size_t)g * HD;
    for (int e = threadIdx.x; e < 8 * RK; e += DEC_THREADS) {
      const int h = e / RK, j = e % RK;
      float acc = 0.f;
      if (h < G) {
        const uint4* qv = reinterpret_cast<const uint4*>(p.q + ((size_t)b * p.n_q + (size_t)g * G + h) * HD);
        const uint4* bv = reinterpret_cast<const uint4*>(Bk + (size_t)j * p.n_kv * HD);
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
      qx[h * RK + j] = __float2bfloat16(acc * p.s_k);
    }
    __syncthreads();
#pragma unroll
    for (int kc = 0; kc < KX; ++kc) {
      qxb[kc][0] = *reinterpret_cast<const uint32_t*>(qx + qrow * RK + kc * 16 + qk);
      qxb[kc][1] = (RK >= 16) ? *reinterpret_cast<const uint32_t*>(qx + qrow * RK + kc * 16 + 8 + qk) : 0u;
    }
  }

  // ---- online-softmax state: this lane's two query columns (2*(lane&3), +1)
  float m0 = NEG_BIG, m1 = NEG_BIG, l0 = 0.f, l1 = 0.f;
  float o[MT + (MX > 0 ? MX : 0)][4];
#pragma unroll
  for (int i = 0; i < MT + MX; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8;   // K' A-operand: row, chunk parity
  const int a_cpar = lane >> 4;
  const int v_row = (lane & 7) + (lane >> 4) * 8;         // V'^T A-operand (transposed load)
  const int v_cpar = (lane >> 3) & 1;

  for (int i = 0; i < my_n; ++i) {
    switch (p.stages) {
      case 2: cp_async_wait<0>(); break;
      case 3: cp_async_wait<1>(); break;
      default: cp_async_wait<2>(); break;
    }
    __syncwarp();                      // tile i visible to all lanes; the slot of tile i-1 is free
    issue_tile(i + p.stages - 1);
    const uint32_t st = ring_u32 + (uint32_t)(i % p.stages) * C::STAGE_BYTES;
    const int t = tile0 + warp + DEC_WARPS * i;
    const int valid = ctx - t * PAGE;   // >= 1; tokens >= valid are masked

    float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kc = 0; kc < KC; ++kc) {
      uint32_t a[4];
      ldsm_x4(a, st + swz_off<CPR_KV>(a_row, 2 * kc + a_cpar));
      mma_bf16_16816(s, a, qb[kc][0], qb[kc][1]);
    }
    if constexpr (RK >= 16) {
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
    if constexpr (RV >= 16) {
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
  }
  cp_async_wait<0>();
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, d);
    l1 += __shfl_xor_sync(0xffffffffu, l1, d);
  }

  // ---- merge the warps of this block: smem [warp][ m[8] | l[8] | O'[OW][8] ]
  __syncthreads();
  float* mg = reinterpret_cast<float*>(smem);
  {
    float* w = mg + warp * (OW * 8 + 16);
    if (lane < 4) { w[2 * lane] = m0; w[2 * lane + 1] = m1; w[8 + 2 * lane] = l0; w[8 + 2 * lane + 1] = l1; }
    const int r = lane >> 2, cq = (lane & 3) * 2;
#pragma unroll
    for (int mt = 0; mt < MT + MX; ++mt) {
      const int row = mt * 16 + r;
      if (row < OW) { w[16 + row * 8 + cq] = o[mt][0]; w[16 + row * 8 + cq + 1] = o[mt][1]; }
      if (row + 8 < OW) { w[16 + (row + 8) * 8 + cq] = o[mt][2]; w[16 + (row + 8) * 8 + cq + 1] = o[mt][3]; }
    }
  }
  __syncthreads();
  // block result, written q-major into the partial record (or kept for the direct epilogue)
  float* rec = p.part + (((size_t)b * p.n_kv + g) * p.max_splits + split) * C::PART_STRIDE;
  __shared__ float fin_m[8], fin_l[8];
  if (threadIdx.x < 8) {
    const int h = threadIdx.x;
    float M = NEG_BIG;
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, mg[w * (OW * 8 + 16) + h]);
    float L = 0.f;
    for (int w = 0; w < DEC_WARPS; ++w) L += mg[w * (OW * 8 + 16) + 8 + h] * fast_exp2(mg[w * (OW * 8 + 16) + h] - M);
    fin_m[h] = M; fin_l[h] = L;
  }
  __syncthreads();
  // fin_o lives behind the per-warp records? no: reuse a separate region after them is not available,
  // so accumulate into registers and write straight to the destination.
  const bool direct = (n_splits == 1);
  float* dst_o = direct ? nullptr : rec + 16;
  // When direct, stage the merged O' in shared memory (region of warp 0 is consumed first, so use a
  // dedicated area placed after all warp records is impossible; instead each thread keeps its values).
  // Element e = h*OW + c handled by thread e % DEC_THREADS.
  constexpr int PER_THREAD = (8 * OW + DEC_THREADS - 1) / DEC_THREADS;
  float acc[PER_THREAD];
#pragma unroll
  for (int k = 0; k < PER_THREAD; ++k) {
    const int e = threadIdx.x + k * DEC_THREADS;
    float v = 0.f;
    if (e < 8 * OW) {
      const int h = e / OW, c = e % OW;
      const float M = fin_m[h];
      for (int w = 0; w < DEC_WARPS; ++w) {
        const float* wr = mg + w * (OW * 8 + 16);
        v += wr[16 + c * 8 + h] * fast_exp2(wr[h] - M);
      }
    }
    acc[k] = v;
  }
  __syncthreads();   // all reads of the warp records are done; smem can be reused
  float* fo = reinterpret_cast<float*>(smem);   // merged O' [8][OW], then m[8], l[8]
  if (!direct) {
#pragma unroll
    for (int k = 0; k < PER_THREAD; ++k) {
      const int e = threadIdx.x + k * DEC_THREADS;
      if (e < 8 * OW) dst_o[e] = acc[k];
    }
    if (threadIdx.x < 8) { rec[threadIdx.x] = fin_m[threadIdx.x]; rec[8 + threadIdx.x] = fin_l[threadIdx.x]; }
    __threadfence();
    __syncthreads();
    __shared__ int is_last;
    if (threadIdx.x == 0) {
      const int old = atomicAdd(p.tickets + (size_t)b * p.n_kv + g, 1);
      is_last = (old == n_splits - 1);
      if (is_last) p.tickets[(size_t)b * p.n_kv + g] = 0;   // ready for the next call
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // merge all splits in split order (deterministic whichever block arrives last)
    const float* base = p.part + (((size_t)b * p.n_kv + g) * p.max_splits) * C::PART_STRIDE;
    if (threadIdx.x < 8) {
      const int h = threadIdx.x;
      float M = NEG_BIG;
      for (int s2 = 0; s2 < n_splits; ++s2) M = fmaxf(M, __ldcg(base + (size_t)s2 * C::PART_STRIDE + h));
      float L = 0.f;
      for (int s2 = 0; s2 < n_splits; ++s2)
        L += __ldcg(base + (size_t)s2 * C::PART_STRIDE + 8 + h) * fast_exp2(__ldcg(base + (size_t)s2 * C::PART_STRIDE + h) - M);
      fin_m[h] = M; fin_l[h] = L;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < PER_THREAD; ++k) {
      const int e = threadIdx.x + k * DEC_THREADS;
      if (e < 8 * OW) {
        const int h = e / OW;
        const float M = fin_m[h];
        float v = 0.f;
        for (int s2 = 0; s2 < n_splits; ++s2) {
          const float* r2 = base + (size_t)s2 * C::PART_STRIDE;
          v += __ldcg(r2 + 16 + e) * fast_exp2(__ldcg(r2 + h) - M);
        }
        fo[e] = v;
      }
    }
  } else {
#pragma unroll
    for (int k = 0; k < PER_THREAD; ++k) {
      const int e = threadIdx.x + k * DEC_THREADS;
      if (e < 8 * OW) fo[e] = acc[k];
    }
  }
  __syncthreads();
  // ---- epilogue: out[h][c] = (O[h][c] + s_v * sum_j U[h][j] * B_v[a][j][g*hd + c]) / l[h]
  const __nv_bfloat16* Bv = RV > 0 ? p.B_v + ((size_t)agent * RV) * ((size_t)p.n_kv * HD) + (size_t)g * HD : nullptr;
  for (int e = threadIdx.x; e < G * HD; e += DEC_THREADS) {
    const int h = e / HD, c = e % HD;
    float v = fo[h * OW + c];
    if constexpr (RV > 0) {
      float u = 0.f;
#pragma unroll 8
      for (int j = 0; j < RV; ++j) u += fo[h * OW + HD + j] * __bfloat162float(Bv[(size_t)j * p.n_kv * HD + c]);
      v += p.s_v * u;
    }
    out_bg[e] = __float2bfloat16(v / fin_l[h]);
  }
}

}  // namespace precc
