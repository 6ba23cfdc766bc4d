// Combine step of context-sharded decode: every shard (a GPU holding a contiguous range of a request's
// tokens) has produced, per (request, kv head), the record of the split-KV merge over its own tokens,
//   rec = [ m[8] | l[8] | O'[G][hd + r_v] ]      (fp32; m in the log2 domain, O' and l relative to m)
// exactly the record the single-GPU ticket kernel keeps per split.  Softmax attention over the union of
// the shards is the same merge once more, followed by the value-side epilogue:
//   M = max_s m_s,  w_s = 2^(m_s - M),  O' = sum_s w_s O'_s,  l = sum_s w_s l_s   (shard order: deterministic)
//   out = (O + s_v U B^V_{a,g}) / l                                   (U = the last r_v columns of O')
// One thread block per (kv head, request); `recs` holds the shards' records back to back,
// [n_shards][B][n_kv][PART_STRIDE], as an all-gather leaves them.
#pragma once
#include "decode.cuh"

namespace precc {

struct CombineParams {
  const float* recs;
  const int32_t* agent_id;
  const __nv_bfloat16* B_v;
  __nv_bfloat16* out;
  uint32_t* status;
  int n_shards, B, n_q, n_kv, group, n_agents;
  float s_v;
};

constexpr int COMBINE_THREADS = 128;

template <int HD, int RV>
__global__ void __launch_bounds__(COMBINE_THREADS)
lr_combine_kernel(const CombineParams p) {
  constexpr int OW = HD + RV;
  constexpr int STRIDE = 8 * OW + 16;                   // DecodeCfg<HD, *, RV>::PART_STRIDE
  __shared__ float w_s[64][8];                          // shard weights per query head
  __shared__ float l_s[8];
  __shared__ float o_s[8 * OW];
  const int g = blockIdx.x, b = blockIdx.y;
  const int G = p.group;
  pdl_wait();
  pdl_launch_dependents();
  const int agent_raw = __ldg(p.agent_id + b);
  const bool use_lr = agent_raw >= 0 && agent_raw < p.n_agents;
  if (agent_raw < -1 || agent_raw >= p.n_agents) { if (threadIdx.x == 0) atomicOr(p.status, StatusBits::BAD_INDEX); }
  const size_t shard_stride = (size_t)p.B * p.n_kv * STRIDE;
  const float* rec0 = p.recs + ((size_t)b * p.n_kv + g) * STRIDE;
  // weights: thread h < G walks the shards of its query head
  if (threadIdx.x < G) {
    const int h = threadIdx.x;
    float M = NEG_BIG;
    for (int s = 0; s < p.n_shards; ++s) M = fmaxf(M, __ldg(rec0 + s * shard_stride + h));
    float L = 0.f;
    for (int s = 0; s < p.n_shards; ++s) {
      const float wv = fast_exp2(__ldg(rec0 + s * shard_stride + h) - M);
      w_s[s][h] = wv;
      L += __ldg(rec0 + s * shard_stride + 8 + h) * wv;
    }
    l_s[h] = L;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < G * OW; e += COMBINE_THREADS) {
    const int h = e / OW;
    float acc = 0.f;
    for (int s = 0; s < p.n_shards; ++s) acc += __ldg(rec0 + s * shard_stride + 16 + e) * w_s[s][h];
    o_s[e] = acc;
  }
  __syncthreads();
  __nv_bfloat16* out_bg = p.out + ((size_t)b * p.n_q + (size_t)g * G) * HD;
  const __nv_bfloat16* Bv = (RV > 0 && use_lr) ? p.B_v + ((size_t)agent_raw * RV) * ((size_t)p.n_kv * HD) + (size_t)g * HD : nullptr;
  for (int e = threadIdx.x; e < G * HD; e += COMBINE_THREADS) {
    const int h = e / HD, c = e % HD;
    float v = o_s[h * OW + c];
    if constexpr (RV > 0) {
      if (use_lr) {
        float u = 0.f;
#pragma unroll 8
        for (int j = 0; j < RV; ++j) u += o_s[h * OW + HD + j] * __bfloat162float(Bv[(size_t)j * p.n_kv * HD + c]);
        v += p.s_v * u;
      }
    }
    const float l = l_s[h];
    out_bg[e] = __float2bfloat16(l > 0.f ? v / l : 0.f);   // no token anywhere: zeros, like an empty context
  }
}

}  // namespace precc
