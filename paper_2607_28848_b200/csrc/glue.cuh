// Element-wise and row-wise pieces of a Llama-3-style decoder layer around the projections (Section 5
// names the model; Section 3.2 has the backward recompute the layer from its saved input): RMSNorm,
// rotary embedding, the SiLU gate, residual add - forward and the input gradients (the base model is
// frozen, so no gradient of the norm gain is produced).  bf16 storage, fp32 arithmetic; all HBM-bound:
// every element is read once and written once with 16-byte accesses.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace mlora {
namespace glue {

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  return make_uint4(ptx::pack_bf16(f[0], f[1]), ptx::pack_bf16(f[2], f[3]), ptx::pack_bf16(f[4], f[5]),
                    ptx::pack_bf16(f[6], f[7]));
}
__device__ __forceinline__ float block_sum(float v, float* red) {      // blockDim.x == 128
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  const float t = red[0] + red[1] + red[2] + red[3];
  __syncthreads();
  return t;
}

// y[t, :] = x[t, :] * rsqrt(mean(x[t, :]^2) + eps) * gain.   One block of 128 threads per row; d % 8 == 0.
__global__ void __launch_bounds__(128)
rmsnorm_fwd_kernel(const __nv_bfloat16* x, int64_t ldx, const float* gain, __nv_bfloat16* y, int64_t ldy, int d, float eps) {
  __shared__ float red[4];
  const __nv_bfloat16* xr = x + (size_t)blockIdx.x * ldx;
  float ss = 0.f;
  for (int k = threadIdx.x * 8; k < d; k += 128 * 8) {
    float f[8];
    unpack8(*reinterpret_cast<const uint4*>(xr + k), f);
#pragma unroll
    for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
  }
  const float rstd = rsqrtf(block_sum(ss, red) / (float)d + eps);
  __nv_bfloat16* yr = y + (size_t)blockIdx.x * ldy;
  for (int k = threadIdx.x * 8; k < d; k += 128 * 8) {
    float f[8];
    unpack8(*reinterpret_cast<const uint4*>(xr + k), f);
    const float4 g0 = *reinterpret_cast<const float4*>(gain + k), g1 = *reinterpret_cast<const float4*>(gain + k + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = f[i] * rstd * g[i];
    *reinterpret_cast<uint4*>(yr + k) = pack8(f);
  }
}

// dx = rstd * (u - xh * mean(u * xh)),  u = gain * dy,  xh = x * rstd  (rstd recomputed from x).
__global__ void __launch_bounds__(128)
rmsnorm_bwd_kernel(const __nv_bfloat16* x, int64_t ldx, const float* gain, const __nv_bfloat16* dy, int64_t lddy,
                   __nv_bfloat16* dx, int64_t lddx, int d, float eps) {
  __shared__ float red[4];
  const __nv_bfloat16* xr = x + (size_t)blockIdx.x * ldx;
  const __nv_bfloat16* dyr = dy + (size_t)blockIdx.x * lddy;
  float ss = 0.f, su = 0.f;
  for (int k = threadIdx.x * 8; k < d; k += 128 * 8) {
    float f[8], g8[8];
    unpack8(*reinterpret_cast<const uint4*>(xr + k), f);
    unpack8(*reinterpret_cast<const uint4*>(dyr + k), g8);
    const float4 g0 = *reinterpret_cast<const float4*>(gain + k), g1 = *reinterpret_cast<const float4*>(gain + k + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) { ss = fmaf(f[i], f[i], ss); su = fmaf(g[i] * g8[i], f[i], su); }
  }
  const float rstd = rsqrtf(block_sum(ss, red) / (float)d + eps);
  const float c = block_sum(su, red) * rstd * rstd / (float)d;          // mean(u * xh) * rstd
  __nv_bfloat16* dxr = dx + (size_t)blockIdx.x * lddx;
  for (int k = threadIdx.x * 8; k < d; k += 128 * 8) {
    float f[8], g8[8], o[8];
    unpack8(*reinterpret_cast<const uint4*>(xr + k), f);
    unpack8(*reinterpret_cast<const uint4*>(dyr + k), g8);
    const float4 g0 = *reinterpret_cast<const float4*>(gain + k), g1 = *reinterpret_cast<const float4*>(gain + k + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = rstd * (g[i] * g8[i] - f[i] * c);
    *reinterpret_cast<uint4*>(dxr + k) = pack8(o);
  }
}

// Rotary embedding of x [T, heads, dh] (row stride ldx elements): elements i and i + dh/2 of a head
// are rotated by pos[t] * theta^(-2i/dh); sign = -1 applies the transposed rotation (the backward).
// One thread per 8 element pairs; dh % 16 == 0.
__global__ void __launch_bounds__(128)
rope_kernel(const __nv_bfloat16* x, int64_t ldx, __nv_bfloat16* y, int64_t ldy, const int32_t* pos, int heads, int dh,
            float log2_theta, float sign) {
  const int t = blockIdx.x;
  const int half = dh / 2, per_head = half / 8;     // 8-pair chunks per head
  const float p = (float)pos[t];
  // a thread owns one chunk of frequencies: their sines and cosines are computed once and used for
  // every head it visits (heads hg, hg + 128 / per_head, ...)
  const int chunk = threadIdx.x % per_head, hg = threadIdx.x / per_head, n_hg = 128 / per_head;
  const int i0 = chunk * 8;
  float sn[8], cs[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float inv = exp2f(-log2_theta * 2.0f * (float)(i0 + i) / (float)dh);
    sincosf(p * inv, &sn[i], &cs[i]);
    sn[i] *= sign;
  }
  for (int h = hg; h < heads; h += n_hg) {
    const __nv_bfloat16* src = x + (size_t)t * ldx + h * dh + i0;
    float a[8], b[8], oa[8], ob[8];
    unpack8(*reinterpret_cast<const uint4*>(src), a);
    unpack8(*reinterpret_cast<const uint4*>(src + half), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      oa[i] = a[i] * cs[i] - b[i] * sn[i];
      ob[i] = b[i] * cs[i] + a[i] * sn[i];
    }
    __nv_bfloat16* dst = y + (size_t)t * ldy + h * dh + i0;
    *reinterpret_cast<uint4*>(dst) = pack8(oa);
    *reinterpret_cast<uint4*>(dst + half) = pack8(ob);
  }
}

// m = silu(g) * u
__global__ void __launch_bounds__(256)
swiglu_fwd_kernel(const __nv_bfloat16* g, const __nv_bfloat16* u, __nv_bfloat16* m, int64_t n8) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    float a[8], b[8], o[8];
    unpack8(reinterpret_cast<const uint4*>(g)[i], a);
    unpack8(reinterpret_cast<const uint4*>(u)[i], b);
#pragma unroll
    for (int k = 0; k < 8; ++k) o[k] = __fdividef(a[k], 1.0f + __expf(-a[k])) * b[k];
    reinterpret_cast<uint4*>(m)[i] = pack8(o);
  }
}

// dg = dm * u * sig(g) * (1 + g * (1 - sig(g))),  du = dm * silu(g)
__global__ void __launch_bounds__(256)
swiglu_bwd_kernel(const __nv_bfloat16* g, const __nv_bfloat16* u, const __nv_bfloat16* dm, __nv_bfloat16* dg,
                  __nv_bfloat16* du, int64_t n8) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    float a[8], b[8], d[8], og[8], ou[8];
    unpack8(reinterpret_cast<const uint4*>(g)[i], a);
    unpack8(reinterpret_cast<const uint4*>(u)[i], b);
    unpack8(reinterpret_cast<const uint4*>(dm)[i], d);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float sg = __fdividef(1.0f, 1.0f + __expf(-a[k]));
      og[k] = d[k] * b[k] * sg * (1.0f + a[k] * (1.0f - sg));
      ou[k] = d[k] * a[k] * sg;
    }
    reinterpret_cast<uint4*>(dg)[i] = pack8(og);
    reinterpret_cast<uint4*>(du)[i] = pack8(ou);
  }
}

// out = a + b
__global__ void __launch_bounds__(256)
add_kernel(const __nv_bfloat16* a, const __nv_bfloat16* b, __nv_bfloat16* out, int64_t n8) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    float x[8], y[8], o[8];
    unpack8(reinterpret_cast<const uint4*>(a)[i], x);
    unpack8(reinterpret_cast<const uint4*>(b)[i], y);
#pragma unroll
    for (int k = 0; k < 8; ++k) o[k] = x[k] + y[k];
    reinterpret_cast<uint4*>(out)[i] = pack8(o);
  }
}

}  // namespace glue
}  // namespace mlora
