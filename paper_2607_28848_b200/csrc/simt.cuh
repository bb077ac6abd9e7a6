// Plain CUDA-core kernels of the multi-LoRA layer, templated on the storage type.  They are the
// product path for fp32 layers (small layers; every product in fp32 FMA) and, for bf16 layers,
// a slow cross-check of the tensor-core kernels that shares none of their index arithmetic.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dropout.cuh"

namespace mlora {
namespace simt {

__device__ __forceinline__ float ld(const float* p) { return *p; }
__device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st(float* p, float v) { *p = v; }
__device__ __forceinline__ void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Out[t, q] = (scale?) * sum_k In[t, k] P_a(t)[q, k]; one warp per (row, q); rows without an
// adapter get zeros, and so do rows whose id lies outside [-1, n_adapters) (the planned path has
// validated its ids on the host; a caller-supplied device table has not been looked at by anyone).  Fine-tuning rows (row_save >= 0) also write u_save (unscaled) and x_save;
// with dropout on, their products skip the dropped columns and count 1 / (1 - p).
template <typename T>
__global__ void shrink_kernel(const T* In, int64_t ld_in, int D, int R, const T* P_all, const float* scale,
                              const int32_t* row_adapter, const int32_t* row_save, float* Out,
                              T* x_save, float* u_save, int64_t save_base, int n_rows, int n_adapters,
                              const DropArgs drop) {
  const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= n_rows * R) return;
  const int t = wid / R, q = wid % R;
  int a = row_adapter[t];
  if (a >= n_adapters) a = -1;
  const int sv = row_save ? row_save[t] : -1;
  float acc = 0.f;
  if (a >= 0) {
    const T* x = In + (size_t)t * ld_in;
    const T* p = P_all + ((size_t)a * R + q) * D;
    if (drop.thr != 0 && sv >= 0) {
      for (int k = lane; k < D; k += 32)
        if (drop_keep(drop, (uint32_t)sv, (uint32_t)k)) acc = fmaf(ld(x + k), ld(p + k), acc);
    } else {
      for (int k = lane; k < D; k += 32) acc = fmaf(ld(x + k), ld(p + k), acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (drop.thr != 0 && sv >= 0) acc *= drop.keep_scale;
  }
  if (lane == 0) {
    Out[(size_t)t * R + q] = (a >= 0 && scale) ? acc * scale[a] : acc;
    if (sv >= 0 && u_save) u_save[(size_t)(save_base + sv) * R + q] = acc;
  }
  if (sv >= 0 && x_save && q == 0) {
    const T* x = In + (size_t)t * ld_in;
    T* d = x_save + (size_t)(save_base + sv) * D;
    for (int k = lane; k < D; k += 32) d[k] = x[k];
  }
}

// Out[m, n] = sum_k In[m, k] Wop(k, n) + sum_q P[m, q] sc L_a(m)[q, n], 32 x 32 tiles.
// W_KMAJOR: Wop(k, n) = W[n * ldw + k]; else Wop(k, n) = W[k * ldw + n].
// With `drop` on (input gradient only) the low-rank term of element (m, n) is kept or dropped
// as the branch input (m, n) was in the forward.
template <typename T, bool W_KMAJOR>
__global__ void gemm_lora_kernel(const T* In, int64_t ld_in, const T* W, int64_t ldw, const T* L_all,
                                 const float* P, const float* scale, const int32_t* row_adapter,
                                 T* Out, int64_t ld_out, int M, int N, int K, int R, int n_adapters,
                                 const DropArgs drop) {
  __shared__ float sIn[32][33];
  __shared__ float sW[32][33];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int m = blockIdx.y * 32 + ty, n = blockIdx.x * 32 + tx;
  float acc = 0.f;
  for (int k0 = 0; k0 < K; k0 += 32) {
    const int mk = blockIdx.y * 32 + ty, kk = k0 + tx;
    sIn[ty][tx] = (mk < M && kk < K) ? ld(In + (size_t)mk * ld_in + kk) : 0.f;
    if (W_KMAJOR) {
      const int nn = blockIdx.x * 32 + ty, kw = k0 + tx;        // sW[n local][k local]
      sW[ty][tx] = (nn < N && kw < K) ? ld(W + (size_t)nn * ldw + kw) : 0.f;
    } else {
      const int kw = k0 + ty, nn = blockIdx.x * 32 + tx;        // sW[k local][n local]
      sW[ty][tx] = (kw < K && nn < N) ? ld(W + (size_t)kw * ldw + nn) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 32; ++k) acc = fmaf(sIn[ty][k], W_KMAJOR ? sW[tx][k] : sW[k][tx], acc);
    __syncthreads();
  }
  if (m < M && n < N) {
    const int a = row_adapter ? row_adapter[m] : -1;
    if (a >= 0 && a < n_adapters) {        // an id outside the adapter tables counts as no adapter
      const float sc = scale ? scale[a] : 1.0f;
      float lo = 0.f;
      for (int q = 0; q < R; ++q) lo = fmaf(P[(size_t)m * R + q], ld(L_all + ((size_t)a * R + q) * N + n), lo);
      if (drop.thr != 0) lo = drop_keep(drop, (uint32_t)m, (uint32_t)n) ? lo * drop.keep_scale : 0.f;
      acc = fmaf(sc, lo, acc);
    }
    st(Out + (size_t)m * ld_out + n, acc);
  }
}

// G[slot, q, j] (+)= sum over the slot's rows of sc P[t, q] Q[t, j]; one thread per (q, j).
// With `drop` on (dA only: Q = the saved branch input) element (t, j) of Q is kept or dropped.
template <typename T>
__global__ void grad_kernel(const float* P, int R, const float* scale, const T* Q, int64_t ldq, int D, float* G,
                            const int32_t* slot_chunk_off, const int32_t* chunk_row0, const int32_t* chunk_nrows,
                            const int32_t* slot_adapter, int accumulate, const DropArgs drop) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int q = blockIdx.y, slot = blockIdx.z;
  if (j >= D) return;
  const float sc = (scale ? scale[slot_adapter[slot]] : 1.0f) * (drop.thr != 0 ? drop.keep_scale : 1.0f);
  float acc = 0.f;
  for (int ch = slot_chunk_off[slot]; ch < slot_chunk_off[slot + 1]; ++ch) {
    const int r0 = chunk_row0[ch], nr = chunk_nrows[ch];
    for (int t = r0; t < r0 + nr; ++t) {
      if (drop.thr != 0 && !drop_keep(drop, (uint32_t)t, (uint32_t)j)) continue;
      acc = fmaf(P[(size_t)t * R + q] * sc, ld(Q + (size_t)t * ldq + j), acc);
    }
  }
  float* dst = G + ((size_t)slot * R + q) * D + j;
  *dst = accumulate ? *dst + acc : acc;
}

// One AdamW update of the adapters of the fine-tuning slots; element i of slot g, rank row q,
// column j.  `which` = blockIdx.y: 0 -> the A matrices (width d_in), 1 -> the B matrices (d_out).
struct AdamwSide {
  const float* grad;   // [n_slots, R, D]
  float* master;       // [n_slots, R, D]
  float* m;
  float* v;
  void* weights;       // [n_adapters, R, D] in the layer's storage type
  int32_t D;
};
struct AdamwArgs {
  AdamwSide side[2];
  const int32_t* slot_adapter;
  int32_t n_slots, R;
  float lr, beta1, beta2, eps, wd, inv_bc1, inv_bc2;   // inv_bc = 1 / (1 - beta^t)
};

template <typename T>
__global__ void adamw_kernel(const AdamwArgs a) {
  const AdamwSide& s = a.side[blockIdx.y];
  const int64_t per_slot = (int64_t)a.R * s.D;
  const int64_t total4 = (int64_t)a.n_slots * per_slot / 4;           // D is a multiple of 4
  for (int64_t i4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i4 < total4; i4 += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = i4 * 4;
    const int slot = (int)(i / per_slot);
    const int64_t off = i - (int64_t)slot * per_slot;
    const float4 g = *reinterpret_cast<const float4*>(s.grad + i);
    float4 w = *reinterpret_cast<const float4*>(s.master + i);
    float4 m = *reinterpret_cast<const float4*>(s.m + i);
    float4 v = *reinterpret_cast<const float4*>(s.v + i);
    float* gw = reinterpret_cast<float*>(const_cast<float4*>(&g));
    float *pw = reinterpret_cast<float*>(&w), *pm = reinterpret_cast<float*>(&m), *pv = reinterpret_cast<float*>(&v);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float wk = pw[k] - a.lr * a.wd * pw[k];
      const float mk = a.beta1 * pm[k] + (1.0f - a.beta1) * gw[k];
      const float vk = a.beta2 * pv[k] + (1.0f - a.beta2) * gw[k] * gw[k];
      wk -= a.lr * (mk * a.inv_bc1) / (sqrtf(vk * a.inv_bc2) + a.eps);
      pw[k] = wk; pm[k] = mk; pv[k] = vk;
    }
    *reinterpret_cast<float4*>(s.master + i) = w;
    *reinterpret_cast<float4*>(s.m + i) = m;
    *reinterpret_cast<float4*>(s.v + i) = v;
    T* dst = reinterpret_cast<T*>(s.weights) + (int64_t)a.slot_adapter[slot] * per_slot + off;
#pragma unroll
    for (int k = 0; k < 4; ++k) st(dst + k, pw[k]);
  }
}

}  // namespace simt
}  // namespace mlora
