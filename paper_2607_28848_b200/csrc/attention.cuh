// Causal softmax attention inside each sequence of a packed batch, grouped-query heads, forward and
// backward, on the CUDA cores: one warp per (row, head); eight keys are in flight per warp (one per
// group of four lanes, each lane holding a quarter of the head dimension) with an online softmax per
// group, the groups being combined at the end.  This is the plain statement of the operation
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

// A warp works on one (row, head).  Its 32 lanes form 8 groups of 4: a group takes every eighth key
// (or query) of the sequence, and inside a group each lane holds a quarter of the head dimension
// (N = dh / 4 consecutive elements), so a dot product costs two shuffles and eight of them run at once.
template <int N>
__device__ __forceinline__ void load_part(const __nv_bfloat16* row, int part, float (&f)[N]) {
  const uint4* p = reinterpret_cast<const uint4*>(row + part * N);
#pragma unroll
  for (int v = 0; v < N / 8; ++v) {
    const uint4 u = p[v];
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[8 * v + 2 * i] = __uint_as_float(w[i] << 16);
      f[8 * v + 2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
}
template <int N>
__device__ __forceinline__ void store_part(__nv_bfloat16* row, int part, const float (&f)[N]) {
  uint4* p = reinterpret_cast<uint4*>(row + part * N);
#pragma unroll
  for (int v = 0; v < N / 8; ++v) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(f[8 * v + 2 * i], f[8 * v + 2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    p[v] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
__device__ __forceinline__ float group_sum(float v) {       // over the 4 lanes of a group
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  return v;
}
__device__ __forceinline__ float across_groups_sum(float v) {   // over the 8 groups, same part
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  v += __shfl_xor_sync(0xffffffffu, v, 8);
  v += __shfl_xor_sync(0xffffffffu, v, 16);
  return v;
}
__device__ __forceinline__ float across_groups_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
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
template <int N>     // N = dh / 4
__global__ void __launch_bounds__(256)
forward_kernel(const AttnArgs a, __nv_bfloat16* o, int64_t ldo, float* lse) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= a.T * a.H) return;
  const int t = w / a.H, h = w % a.H, hk = h / (a.H / a.Hkv);
  const int grp = lane >> 2, part = lane & 3, dh = 4 * N;
  float q[N], acc[N];
  load_part<N>(a.q + (size_t)t * a.ldq + h * dh, part, q);
#pragma unroll
  for (int e = 0; e < N; ++e) { q[e] *= a.scale; acc[e] = 0.f; }
  float m = -INFINITY, l = 0.f;                      // this group's running maximum and sum
  for (int j0 = a.seq_start[t]; j0 <= t; j0 += 8) {
    const int j = j0 + grp;
    if (j <= t) {                                     // uniform inside a group: its shuffles stay inside it
      float kk[N], vv[N];
      load_part<N>(a.k + (size_t)j * a.ldk + hk * dh, part, kk);
      load_part<N>(a.v + (size_t)j * a.ldv + hk * dh, part, vv);
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < N; ++e) s = fmaf(q[e], kk[e], s);
      s += __shfl_xor_sync(0xfu << (4 * grp), s, 1);
      s += __shfl_xor_sync(0xfu << (4 * grp), s, 2);
      const float m2 = fmaxf(m, s);
      const float c = __expf(m - m2), p = __expf(s - m2);
      l = l * c + p;
#pragma unroll
      for (int e = 0; e < N; ++e) acc[e] = acc[e] * c + p * vv[e];
      m = m2;
    }
  }
  // combine the 8 groups (a group without keys has m = -inf, l = 0 and contributes nothing)
  const float M = across_groups_max(m);
  const float f = (m == -INFINITY) ? 0.f : __expf(m - M);
  const float L = across_groups_sum(l * f);
  const float inv = 1.0f / L;
#pragma unroll
  for (int e = 0; e < N; ++e) acc[e] = across_groups_sum(acc[e] * f) * inv;
  if (grp == 0) store_part<N>(o + (size_t)t * ldo + h * dh, part, acc);
  if (lane == 0) lse[(size_t)t * a.H + h] = M + __logf(L);
}

// dQ: warp = (row t, head h)
template <int N>
__global__ void __launch_bounds__(256)
backward_dq_kernel(const AttnArgs a, const __nv_bfloat16* o, int64_t ldo, const float* lse, const __nv_bfloat16* dO,
                   int64_t lddo, __nv_bfloat16* dq, int64_t lddq) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= a.T * a.H) return;
  const int t = w / a.H, h = w % a.H, hk = h / (a.H / a.Hkv);
  const int grp = lane >> 2, part = lane & 3, dh = 4 * N;
  float q[N], g[N], acc[N];
  {
    float oo[N];
    load_part<N>(a.q + (size_t)t * a.ldq + h * dh, part, q);
    load_part<N>(dO + (size_t)t * lddo + h * dh, part, g);
    load_part<N>(o + (size_t)t * ldo + h * dh, part, oo);
    float d = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) { d = fmaf(g[e], oo[e], d); acc[e] = 0.f; }
    d = group_sum(d);                  // D_i = dO_i . o_i, the same in every group
    const float D = d;
    const float L = lse[(size_t)t * a.H + h];
    for (int j0 = a.seq_start[t]; j0 <= t; j0 += 8) {
      const int j = j0 + grp;
      if (j <= t) {
        float kk[N], vv[N];
        load_part<N>(a.k + (size_t)j * a.ldk + hk * dh, part, kk);
        load_part<N>(a.v + (size_t)j * a.ldv + hk * dh, part, vv);
        float s = 0.f, dp = 0.f;
#pragma unroll
        for (int e = 0; e < N; ++e) { s = fmaf(q[e], kk[e], s); dp = fmaf(g[e], vv[e], dp); }
        const unsigned gm = 0xfu << (4 * grp);
        s += __shfl_xor_sync(gm, s, 1); s += __shfl_xor_sync(gm, s, 2);
        dp += __shfl_xor_sync(gm, dp, 1); dp += __shfl_xor_sync(gm, dp, 2);
        const float ds = __expf(s * a.scale - L) * (dp - D) * a.scale;
#pragma unroll
        for (int e = 0; e < N; ++e) acc[e] = fmaf(ds, kk[e], acc[e]);
      }
    }
  }
#pragma unroll
  for (int e = 0; e < N; ++e) acc[e] = across_groups_sum(acc[e]);
  if (grp == 0) store_part<N>(dq + (size_t)t * lddq + h * dh, part, acc);
}

// dK, dV: warp = (key row j, kv head hk); sums over the later rows of the sequence (eight at a time, one per
// group) and the query heads of hk
template <int N>
__global__ void __launch_bounds__(256)
backward_dkv_kernel(const AttnArgs a, const __nv_bfloat16* o, int64_t ldo, const float* lse, const __nv_bfloat16* dO,
                    int64_t lddo, __nv_bfloat16* dk, int64_t lddk, __nv_bfloat16* dv, int64_t lddv) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= a.T * a.Hkv) return;
  const int j = w / a.Hkv, hk = w % a.Hkv, rep = a.H / a.Hkv;
  const int grp = lane >> 2, part = lane & 3, dh = 4 * N;
  float kk[N], vv[N], ak[N], av[N];
  load_part<N>(a.k + (size_t)j * a.ldk + hk * dh, part, kk);
  load_part<N>(a.v + (size_t)j * a.ldv + hk * dh, part, vv);
#pragma unroll
  for (int e = 0; e < N; ++e) ak[e] = av[e] = 0.f;
  const int end = a.seq_end[j];
  for (int i0 = j; i0 < end; i0 += 8) {
    const int i = i0 + grp;
    if (i < end) {
      const unsigned gm = 0xfu << (4 * grp);
      for (int r = 0; r < rep; ++r) {
        const int h = hk * rep + r;
        float q[N], g[N], oo[N];
        load_part<N>(a.q + (size_t)i * a.ldq + h * dh, part, q);
        load_part<N>(dO + (size_t)i * lddo + h * dh, part, g);
        load_part<N>(o + (size_t)i * ldo + h * dh, part, oo);
        float s = 0.f, dp = 0.f, D = 0.f;
#pragma unroll
        for (int e = 0; e < N; ++e) { s = fmaf(q[e], kk[e], s); dp = fmaf(g[e], vv[e], dp); D = fmaf(g[e], oo[e], D); }
        s += __shfl_xor_sync(gm, s, 1); s += __shfl_xor_sync(gm, s, 2);
        dp += __shfl_xor_sync(gm, dp, 1); dp += __shfl_xor_sync(gm, dp, 2);
        D += __shfl_xor_sync(gm, D, 1); D += __shfl_xor_sync(gm, D, 2);
        const float p = __expf(s * a.scale - lse[(size_t)i * a.H + h]);
        const float ds = p * (dp - D) * a.scale;
#pragma unroll
        for (int e = 0; e < N; ++e) { ak[e] = fmaf(ds, q[e], ak[e]); av[e] = fmaf(p, g[e], av[e]); }
      }
    }
  }
#pragma unroll
  for (int e = 0; e < N; ++e) { ak[e] = across_groups_sum(ak[e]); av[e] = across_groups_sum(av[e]); }
  if (grp == 0) {
    store_part<N>(dk + (size_t)j * lddk + hk * dh, part, ak);
    store_part<N>(dv + (size_t)j * lddv + hk * dh, part, av);
  }
}

}  // namespace attn
}  // namespace mlora
