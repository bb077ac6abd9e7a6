// Causal softmax attention inside each sequence of a packed batch, grouped-query heads, forward and
// backward, on the CUDA cores: one warp per (row, head), the head dimension spread over the lanes,
// keys visited one at a time with an online softmax.  This is the plain statement of the operation
// for the decoder-layer module (fine-tuning sequences of a few hundred tokens), not a tensor-core
// flash kernel: the layer's hot operations are the projections.
//   s_ij = q_i . k_j / sqrt(dh)  (j <= i, same sequence),  p_ij = softmax_j(s_ij),  o_i = sum_j p_ij v_j
//   backward: D_i = dO_i . o_i;  dS_ij = p_ij (dO_i . v_j - D_i);  dQ_i = sum_j dS_ij k_j / sqrt(dh);
//             dK_j = sum_i dS_ij q_i / sqrt(dh);  dV_j = sum_i p_ij dO_i   (sums over the query heads of a kv head too)
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mlora {
namespace attn {

template <int E>   // elements of the head dimension per lane: dh = 32 E
__device__ __forceinline__ void load_row(const __nv_bfloat16* p, int lane, float (&f)[E]) {
#pragma unroll
  for (int e = 0; e < E; ++e) f[e] = __bfloat162float(p[lane + 32 * e]);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

struct AttnArgs {
  const __nv_bfloat16 *q, *k, *v;     // q [T, H, dh]; k, v [T, Hkv, dh]
  int64_t ldq, ldk, ldv;              // row strides in elements
  const int32_t* seq_start;           // [T] first row of the row's sequence
  const int32_t* seq_end;             // [T] one past the last row of the row's sequence
  int32_t T, H, Hkv;
  float scale;                        // 1 / sqrt(dh)
};

// grid: ceil(T * H / 8) blocks of 8 warps; warp = (row t, head h)
template <int E>
__global__ void __launch_bounds__(256)
forward_kernel(const AttnArgs a, __nv_bfloat16* o, int64_t ldo, float* lse) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= a.T * a.H) return;
  const int t = w / a.H, h = w % a.H, hk = h / (a.H / a.Hkv);
  float q[E], acc[E];
  load_row<E>(a.q + (size_t)t * a.ldq + h * 32 * E, lane, q);
#pragma unroll
  for (int e = 0; e < E; ++e) { q[e] *= a.scale; acc[e] = 0.f; }
  float m = -INFINITY, l = 0.f;
  for (int j = a.seq_start[t]; j <= t; ++j) {
    float kk[E], vv[E];
    load_row<E>(a.k + (size_t)j * a.ldk + hk * 32 * E, lane, kk);
    load_row<E>(a.v + (size_t)j * a.ldv + hk * 32 * E, lane, vv);
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) s = fmaf(q[e], kk[e], s);
    s = warp_sum(s);
    const float m2 = fmaxf(m, s);
    const float c = __expf(m - m2), p = __expf(s - m2);
    l = l * c + p;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * c + p * vv[e];
    m = m2;
  }
  const float inv = 1.0f / l;
#pragma unroll
  for (int e = 0; e < E; ++e) o[(size_t)t * ldo + h * 32 * E + lane + 32 * e] = __float2bfloat16_rn(acc[e] * inv);
  if (lane == 0) lse[(size_t)t * a.H + h] = m + __logf(l);
}

// dQ: warp = (row t, head h)
template <int E>
__global__ void __launch_bounds__(256)
backward_dq_kernel(const AttnArgs a, const __nv_bfloat16* o, int64_t ldo, const float* lse, const __nv_bfloat16* dO,
                   int64_t lddo, __nv_bfloat16* dq, int64_t lddq) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= a.T * a.H) return;
  const int t = w / a.H, h = w % a.H, hk = h / (a.H / a.Hkv);
  float q[E], g[E], oo[E], acc[E];
  load_row<E>(a.q + (size_t)t * a.ldq + h * 32 * E, lane, q);
  load_row<E>(dO + (size_t)t * lddo + h * 32 * E, lane, g);
  load_row<E>(o + (size_t)t * ldo + h * 32 * E, lane, oo);
  float D = 0.f;
#pragma unroll
  for (int e = 0; e < E; ++e) { D = fmaf(g[e], oo[e], D); acc[e] = 0.f; }
  D = warp_sum(D);
  const float L = lse[(size_t)t * a.H + h];
  for (int j = a.seq_start[t]; j <= t; ++j) {
    float kk[E], vv[E];
    load_row<E>(a.k + (size_t)j * a.ldk + hk * 32 * E, lane, kk);
    load_row<E>(a.v + (size_t)j * a.ldv + hk * 32 * E, lane, vv);
    float s = 0.f, dp = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) { s = fmaf(q[e], kk[e], s); dp = fmaf(g[e], vv[e], dp); }
    s = warp_sum(s) * a.scale;
    dp = warp_sum(dp);
    const float ds = __expf(s - L) * (dp - D) * a.scale;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = fmaf(ds, kk[e], acc[e]);
  }
#pragma unroll
  for (int e = 0; e < E; ++e) dq[(size_t)t * lddq + h * 32 * E + lane + 32 * e] = __float2bfloat16_rn(acc[e]);
}

// dK, dV: warp = (key row j, kv head hk); sums over the later rows of the sequence and the query heads of hk
template <int E>
__global__ void __launch_bounds__(256)
backward_dkv_kernel(const AttnArgs a, const __nv_bfloat16* o, int64_t ldo, const float* lse, const __nv_bfloat16* dO,
                    int64_t lddo, __nv_bfloat16* dk, int64_t lddk, __nv_bfloat16* dv, int64_t lddv) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= a.T * a.Hkv) return;
  const int j = w / a.Hkv, hk = w % a.Hkv, rep = a.H / a.Hkv;
  float kk[E], vv[E], ak[E], av[E];
  load_row<E>(a.k + (size_t)j * a.ldk + hk * 32 * E, lane, kk);
  load_row<E>(a.v + (size_t)j * a.ldv + hk * 32 * E, lane, vv);
#pragma unroll
  for (int e = 0; e < E; ++e) ak[e] = av[e] = 0.f;
  for (int i = j; i < a.seq_end[j]; ++i) {
    for (int r = 0; r < rep; ++r) {
      const int h = hk * rep + r;
      float q[E], g[E], oo[E];
      load_row<E>(a.q + (size_t)i * a.ldq + h * 32 * E, lane, q);
      load_row<E>(dO + (size_t)i * lddo + h * 32 * E, lane, g);
      load_row<E>(o + (size_t)i * ldo + h * 32 * E, lane, oo);
      float s = 0.f, dp = 0.f, D = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) { s = fmaf(q[e], kk[e], s); dp = fmaf(g[e], vv[e], dp); D = fmaf(g[e], oo[e], D); }
      s = warp_sum(s) * a.scale;
      dp = warp_sum(dp);
      D = warp_sum(D);
      const float p = __expf(s - lse[(size_t)i * a.H + h]);
      const float ds = p * (dp - D) * a.scale;
#pragma unroll
      for (int e = 0; e < E; ++e) { ak[e] = fmaf(ds, q[e], ak[e]); av[e] = fmaf(p, g[e], av[e]); }
    }
  }
#pragma unroll
  for (int e = 0; e < E; ++e) {
    dk[(size_t)j * lddk + hk * 32 * E + lane + 32 * e] = __float2bfloat16_rn(ak[e]);
    dv[(size_t)j * lddv + hk * 32 * E + lane + 32 * e] = __float2bfloat16_rn(av[e]);
  }
}

}  // namespace attn
}  // namespace mlora
