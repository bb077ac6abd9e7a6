// Rank-r ("skinny") kernels of the multi-LoRA layer for bf16 storage.  Both are bound by the
// bytes of the wide operand they stream once from HBM; the rank-r contraction itself runs on the
// warp-level tensor-core instruction (mma.sync m16n8k16, fp32 accumulate) because at rank 16 and
// above the CUDA cores could not keep up with the memory system.
//
//  shrink_kernel : Out[t, q] = sum_k In[t, k] * P_a(t)[q, k]      (U = X A^T  and  V = s dY B^T)
//                  work item = up to 16 consecutive rows bound to one adapter (a decode row is an
//                  item of one row: the gather-by-adapter-id case); optionally copies the rows of
//                  In and the result into the fine-tuning activation buffers on the way.
//  grad_kernel   : G_g[q, j] = sum_{rows t of slot g} P[t, q] * Q[t, j]   (dB = (s U)^T dY, dA = V^T X)
#pragma once

#include "ptx.cuh"

namespace mlora {

constexpr int SHRINK_THREADS = 128;
constexpr int GRAD_THREADS = 256;

struct ShrinkArgs {
  const __nv_bfloat16* In;     // [rows, D], row stride ld_in
  int64_t ld_in;
  int32_t D;                   // multiple of 64
  const __nv_bfloat16* P_all;  // [n_adapters, R, D]
  const float* scale;          // nullable: result multiplied by scale[adapter]
  float* Out;                  // [rows, R]
  const int32_t* item_row0;
  const int32_t* item_nrows;
  const int32_t* item_adapter;
  const int32_t* item_save0;   // nullable
  __nv_bfloat16* x_save;       // nullable, [cap, D] dense
  float* u_save;               // nullable, [cap, R] dense
  int64_t save_base;
};

// One CTA per item; its 4 warps take the 64-wide K blocks round-robin and reduce through shared
// memory.  Operand fragments come straight from global memory as 16-byte loads: within a K block
// thread (g, c) of a warp reads elements 16c .. 16c+15 of rows g and g+8, and the same elements
// of the adapter rows; since the contraction index may be permuted freely (identically on both
// operands) these 16 consecutive elements are used as the thread's share of 4 MMA steps.
template <int RB>   // RB = R / 8 column blocks of the m16n8k16 MMA
__global__ void __launch_bounds__(SHRINK_THREADS)
shrink_kernel(const ShrinkArgs a) {
  constexpr int R = RB * 8;
  constexpr int NBG = RB < 4 ? RB : 4;           // column blocks processed together
  __shared__ float red[4][16][R + 1];

  const int item = blockIdx.x;
  const int row0 = a.item_row0[item];
  const int nrows = a.item_nrows[item];
  const int adapter = a.item_adapter[item];
  const int save0 = a.item_save0 ? a.item_save0[item] : -1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const bool v0 = g < nrows, v1 = g + 8 < nrows;
  const __nv_bfloat16* x0 = a.In + (size_t)(row0 + g) * a.ld_in + 16 * c;
  const __nv_bfloat16* x1 = a.In + (size_t)(row0 + g + 8) * a.ld_in + 16 * c;
  const __nv_bfloat16* p0 = a.P_all + ((size_t)adapter * R + g) * a.D + 16 * c;
  __nv_bfloat16* s0 = nullptr;
  __nv_bfloat16* s1 = nullptr;
  if (save0 >= 0 && a.x_save) {
    s0 = a.x_save + (size_t)(a.save_base + save0 + g) * a.D + 16 * c;
    s1 = a.x_save + (size_t)(a.save_base + save0 + g + 8) * a.D + 16 * c;
  }

  float acc[RB][4];
#pragma unroll
  for (int i = 0; i < RB; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

  const int nkb = a.D / 64;
  const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll 2
  for (int kb = warp; kb < nkb; kb += 4) {
    const int ko = kb * 64;
    uint4 xa0 = zero4, xa1 = zero4, xb0 = zero4, xb1 = zero4;
    if (v0) { xa0 = ptx::ldg_nc_v4(x0 + ko); xa1 = ptx::ldg_nc_v4(x0 + ko + 8); }
    if (v1) { xb0 = ptx::ldg_nc_v4(x1 + ko); xb1 = ptx::ldg_nc_v4(x1 + ko + 8); }
    const uint32_t ra[8] = {xa0.x, xa0.y, xa0.z, xa0.w, xa1.x, xa1.y, xa1.z, xa1.w};
    const uint32_t rb[8] = {xb0.x, xb0.y, xb0.z, xb0.w, xb1.x, xb1.y, xb1.z, xb1.w};
#pragma unroll
    for (int nb0 = 0; nb0 < RB; nb0 += NBG) {
      uint4 pa[NBG], pb[NBG];
#pragma unroll
      for (int i = 0; i < NBG; ++i) {
        const __nv_bfloat16* pp = p0 + (size_t)(nb0 + i) * 8 * a.D + ko;
        pa[i] = __ldg(reinterpret_cast<const uint4*>(pp));
        pb[i] = __ldg(reinterpret_cast<const uint4*>(pp + 8));
      }
#pragma unroll
      for (int i = 0; i < NBG; ++i) {
        const uint32_t rp[8] = {pa[i].x, pa[i].y, pa[i].z, pa[i].w, pb[i].x, pb[i].y, pb[i].z, pb[i].w};
#pragma unroll
        for (int s = 0; s < 4; ++s)
          ptx::mma_bf16_16816(acc[nb0 + i], ra[2 * s], rb[2 * s], ra[2 * s + 1], rb[2 * s + 1], rp[2 * s], rp[2 * s + 1]);
      }
    }
    if (s0) {     // activation save: the rows of In pass through registers exactly once
      if (v0) { *reinterpret_cast<uint4*>(s0 + ko) = xa0; *reinterpret_cast<uint4*>(s0 + ko + 8) = xa1; }
      if (v1) { *reinterpret_cast<uint4*>(s1 + ko) = xb0; *reinterpret_cast<uint4*>(s1 + ko + 8) = xb1; }
    }
  }

#pragma unroll
  for (int i = 0; i < RB; ++i) {
    red[warp][g][i * 8 + 2 * c] = acc[i][0];
    red[warp][g][i * 8 + 2 * c + 1] = acc[i][1];
    red[warp][g + 8][i * 8 + 2 * c] = acc[i][2];
    red[warp][g + 8][i * 8 + 2 * c + 1] = acc[i][3];
  }
  __syncthreads();
  const float sc = a.scale ? a.scale[adapter] : 1.0f;
  for (int idx = threadIdx.x; idx < nrows * R; idx += SHRINK_THREADS) {
    const int r = idx / R, q = idx % R;
    const float u = (red[0][r][q] + red[1][r][q]) + (red[2][r][q] + red[3][r][q]);
    a.Out[(size_t)(row0 + r) * R + q] = u * sc;
    if (save0 >= 0 && a.u_save) a.u_save[(size_t)(a.save_base + save0 + r) * R + q] = u;
  }
}

struct GradArgs {
  const float* P;              // [rows, R] fp32
  int32_t R;
  const float* scale;          // nullable: P multiplied by scale[slot_adapter[slot]]
  const __nv_bfloat16* Q;      // [rows, D], row stride ldq
  int64_t ldq;
  int32_t D;                   // multiple of 64
  float* G;                    // [n_slots, R, D]
  const int32_t* slot_chunk_off;
  const int32_t* chunk_row0;
  const int32_t* chunk_nrows;
  const int32_t* slot_adapter;
  int32_t accumulate;
};

// grid = (D / 64, n_slots, ceil(R / (16 MB))).  A CTA owns a 64-column strip of one slot's
// gradient (and MB blocks of 16 rank rows); its 8 warps share the slot's row chunks, each
// accumulating G^T-style with the rows as the MMA's contraction index, and are summed in a fixed
// order, so the result does not depend on scheduling.  P is split into a bf16 head and a bf16
// remainder (two MMAs) to keep ~16 bits of its mantissa.
template <int MB>
__global__ void __launch_bounds__(GRAD_THREADS)
grad_kernel(const GradArgs a) {
  __shared__ float red[MB * 16][64 + 1];
  const int slot = blockIdx.y;
  const int j0 = blockIdx.x * 64;
  const int qbase = blockIdx.z * MB * 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const float sc = a.scale ? a.scale[a.slot_adapter[slot]] : 1.0f;
  const int R = a.R;

  float acc[MB][8][4];
#pragma unroll
  for (int m = 0; m < MB; ++m)
#pragma unroll
    for (int n = 0; n < 8; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;

  const int ch0 = a.slot_chunk_off[slot], ch1 = a.slot_chunk_off[slot + 1];
  const uint4 zero4 = make_uint4(0, 0, 0, 0);
  const int tr[4] = {2 * c, 2 * c + 1, 2 * c + 8, 2 * c + 9};
#pragma unroll 2
  for (int ch = ch0 + warp; ch < ch1; ch += GRAD_THREADS / 32) {
    const int row0 = a.chunk_row0[ch], nrows = a.chunk_nrows[ch];
    uint4 q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      q[i] = tr[i] < nrows ? ptx::ldg_nc_v4(a.Q + (size_t)(row0 + tr[i]) * a.ldq + j0 + 8 * g) : zero4;
    uint32_t ahi[MB][4], alo[MB][4];
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      float pv[4][2];     // [row index][q = g / g + 8]
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int qq = qbase + m * 16 + g + 8 * h;
          pv[i][h] = (tr[i] < nrows && qq < R) ? __ldg(a.P + (size_t)(row0 + tr[i]) * R + qq) * sc : 0.f;
        }
      }
      // fragment order: a0 (q=g, rows 2c,2c+1), a1 (q=g+8, rows 2c,2c+1), a2 (q=g, rows 2c+8,2c+9), a3
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const int h = f & 1, rp = (f >> 1) * 2;
        const float e0 = pv[rp][h], e1 = pv[rp + 1][h];
        const __nv_bfloat16 h0 = __float2bfloat16_rn(e0), h1 = __float2bfloat16_rn(e1);
        ahi[m][f] = ptx::pack_bf16(e0, e1);
        alo[m][f] = ptx::pack_bf16(e0 - __bfloat162float(h0), e1 - __bfloat162float(h1));
      }
    }
    const uint32_t qr[4][4] = {{q[0].x, q[0].y, q[0].z, q[0].w}, {q[1].x, q[1].y, q[1].z, q[1].w},
                               {q[2].x, q[2].y, q[2].z, q[2].w}, {q[3].x, q[3].y, q[3].z, q[3].w}};
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      const uint32_t sel = (nb & 1) ? 0x7632u : 0x5410u;
      const uint32_t b0 = __byte_perm(qr[0][nb >> 1], qr[1][nb >> 1], sel);
      const uint32_t b1 = __byte_perm(qr[2][nb >> 1], qr[3][nb >> 1], sel);
#pragma unroll
      for (int m = 0; m < MB; ++m) {
        ptx::mma_bf16_16816(acc[m][nb], ahi[m][0], ahi[m][1], ahi[m][2], ahi[m][3], b0, b1);
        ptx::mma_bf16_16816(acc[m][nb], alo[m][0], alo[m][1], alo[m][2], alo[m][3], b0, b1);
      }
    }
  }

  // fixed-order sum over the warps; column block nb, MMA column n  <->  strip column 8 n + nb
  for (int w = 0; w < GRAD_THREADS / 32; ++w) {
    if (warp == w) {
#pragma unroll
      for (int m = 0; m < MB; ++m)
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
          float* r0 = &red[m * 16 + g][0];
          float* r1 = &red[m * 16 + g + 8][0];
          const int ca = 8 * (2 * c) + nb, cb = 8 * (2 * c + 1) + nb;
          if (w == 0) { r0[ca] = acc[m][nb][0]; r0[cb] = acc[m][nb][1]; r1[ca] = acc[m][nb][2]; r1[cb] = acc[m][nb][3]; }
          else        { r0[ca] += acc[m][nb][0]; r0[cb] += acc[m][nb][1]; r1[ca] += acc[m][nb][2]; r1[cb] += acc[m][nb][3]; }
        }
    }
    __syncthreads();
  }
  for (int idx = threadIdx.x; idx < MB * 16 * 64; idx += GRAD_THREADS) {
    const int ql = idx / 64, j = idx % 64;
    const int qq = qbase + ql;
    if (qq >= R) continue;
    float* dst = a.G + ((size_t)slot * R + qq) * a.D + j0 + j;
    *dst = a.accumulate ? (*dst + red[ql][j]) : red[ql][j];
  }
}

}  // namespace mlora
