// Rank-r ("skinny") kernels of the multi-LoRA layer for bf16 storage.  Both are bound by the
// bytes of the wide operand they stream once from HBM; the rank-r contraction itself runs on the
// warp-level tensor-core instruction (mma.sync m16n8k16, fp32 accumulate) because at rank 16 and
// above the CUDA cores could not keep up with the memory system.
//
//  shrink_kernel : Out[t, q] = sum_k In[t, k] * P_a(t)[q, k]      (U = X A^T  and  V = s dY B^T)
//                  work item = up to 32 rows that share one adapter, GATHERED by adapter id (they
//                  need not be adjacent: decode rows of one adapter form one item, prefill and
//                  fine-tune segments are runs of items); optionally copies the rows of In and the
//                  result into the fine-tuning activation buffers on the way.
//  grad_kernel   : G_g[q, j] = sum_{rows t of slot g} P[t, q] * Q[t, j]   (dB = (s U)^T dY, dA = V^T X)
#pragma once

#include "ptx.cuh"

namespace mlora {

constexpr int GRAD_THREADS = 256;

struct ShrinkArgs {
  const __nv_bfloat16* In;     // [rows, D], row stride ld_in
  int64_t ld_in;
  int32_t D;                   // multiple of 64
  const __nv_bfloat16* P_all;  // [n_adapters, R, D]
  const float* scale;          // nullable: result multiplied by scale[adapter]
  float* Out;                  // [rows, R]
  const int32_t* item_rows;    // row ids grouped by adapter
  const int32_t* item_start;   // first entry of the item in item_rows
  const int32_t* item_nrows;
  const int32_t* item_adapter;
  const int32_t* row_save;     // nullable: [rows] save offset of a row or -1
  __nv_bfloat16* x_save;       // nullable, [cap, D] dense
  float* u_save;               // nullable, [cap, R] dense
  int64_t save_base;
  // split of the contraction over gridDim.y CTAs per item (used when there are few items):
  float* partial;              // [n_items * gridDim.z * gridDim.y, MT * 16, R] scratch
  int32_t* counters;           // [n_items * gridDim.z], zero between launches
};

// One CTA per item; its warps take the 64-wide K blocks round-robin and reduce through shared
// memory.  Operand fragments come straight from global memory as 16-byte loads: within a K block
// thread (g, c) of a warp reads elements 16c .. 16c+15 of rows g, g+8 (, g+16, g+24) of the item
// and the same elements of the adapter rows; since the contraction index may be permuted freely
// (identically on both operands) these 16 consecutive elements are used as the thread's share of
// 4 MMA steps.  RB = R / 8 column blocks, MT = 16-row blocks per item, WARPS = warps per CTA.
// With gridDim.y > 1 the K range of an item is split over that many CTAs; each leaves its partial
// result in scratch and the CTA that finishes last adds them up in a fixed order, so the result
// does not depend on which CTA that was.
template <int RB, int MT, int WARPS, int MIN_CTAS>
__global__ void __launch_bounds__(WARPS * 32, MIN_CTAS)
shrink_kernel(const ShrinkArgs a) {
  constexpr int R = RB * 8;
  constexpr int NBG = RB < 4 ? RB : 4;           // column blocks processed together
  __shared__ float red[WARPS][MT * 16][R + 1];

  // gridDim.z = 32 / (16 MT) CTAs share the rows of a plan item when MT covers only part of it
  const int roff = blockIdx.z * MT * 16;
  const int nrows_item = a.item_nrows[blockIdx.x] - roff;
  if (nrows_item <= 0) return;
  const int nrows = nrows_item < MT * 16 ? nrows_item : MT * 16;
  const int item = blockIdx.x * gridDim.z + blockIdx.z;          // index of this row block in the scratch
  const int adapter = a.item_adapter[blockIdx.x];
  const int32_t* rows = a.item_rows + a.item_start[blockIdx.x] + roff;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  // this thread's rows: local index g + 8 j, j < 2 MT
  const __nv_bfloat16* xp[2 * MT];
  __nv_bfloat16* sp[2 * MT];
#pragma unroll
  for (int j = 0; j < 2 * MT; ++j) {
    const int rl = g + 8 * j;
    xp[j] = nullptr; sp[j] = nullptr;
    if (rl < nrows) {
      const int row = rows[rl];
      xp[j] = a.In + (size_t)row * a.ld_in + 16 * c;
      const int sv = (a.row_save && a.x_save) ? a.row_save[row] : -1;
      if (sv >= 0) sp[j] = a.x_save + (size_t)(a.save_base + sv) * a.D + 16 * c;
    }
  }
  const __nv_bfloat16* p0 = a.P_all + ((size_t)adapter * R + g) * a.D + 16 * c;

  float acc[MT][RB][4];
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int i = 0; i < RB; ++i) acc[m][i][0] = acc[m][i][1] = acc[m][i][2] = acc[m][i][3] = 0.f;

  const int nkb = a.D / 64;
  const int ksplit = gridDim.y, ks = blockIdx.y;
  const int kb_begin = (int)((long long)ks * nkb / ksplit), kb_end = (int)((long long)(ks + 1) * nkb / ksplit);
  const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll 2
  for (int kb = kb_begin + warp; kb < kb_end; kb += WARPS) {
    const int ko = kb * 64;
    uint4 x[2 * MT][2];
#pragma unroll
    for (int j = 0; j < 2 * MT; ++j) {
      x[j][0] = zero4; x[j][1] = zero4;
      if (xp[j]) { x[j][0] = ptx::ldg_nc_v4(xp[j] + ko); x[j][1] = ptx::ldg_nc_v4(xp[j] + ko + 8); }
    }
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
        for (int m = 0; m < MT; ++m) {
          const uint4 &l0 = x[2 * m][0], &l1 = x[2 * m][1], &h0 = x[2 * m + 1][0], &h1 = x[2 * m + 1][1];
          const uint32_t ra[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
          const uint32_t rb[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
#pragma unroll
          for (int s = 0; s < 4; ++s)
            ptx::mma_bf16_16816(acc[m][nb0 + i], ra[2 * s], rb[2 * s], ra[2 * s + 1], rb[2 * s + 1], rp[2 * s],
                                rp[2 * s + 1]);
        }
      }
    }
    // activation save: the rows of In pass through registers exactly once
#pragma unroll
    for (int j = 0; j < 2 * MT; ++j)
      if (sp[j]) {
        *reinterpret_cast<uint4*>(sp[j] + ko) = x[j][0];
        *reinterpret_cast<uint4*>(sp[j] + ko + 8) = x[j][1];
      }
  }

#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      red[warp][m * 16 + g][i * 8 + 2 * c] = acc[m][i][0];
      red[warp][m * 16 + g][i * 8 + 2 * c + 1] = acc[m][i][1];
      red[warp][m * 16 + g + 8][i * 8 + 2 * c] = acc[m][i][2];
      red[warp][m * 16 + g + 8][i * 8 + 2 * c + 1] = acc[m][i][3];
    }
  __syncthreads();
  const float sc = a.scale ? a.scale[adapter] : 1.0f;
  __shared__ int is_last;
  if (ksplit > 1) {
    float* mine = a.partial + ((size_t)item * ksplit + ks) * (MT * 16 * R);
    for (int idx = threadIdx.x; idx < nrows * R; idx += WARPS * 32) {
      const int r = idx / R, q = idx % R;
      float u = 0.f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) u += red[w][r][q];
      mine[idx] = u;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(a.counters + item, 1) == ksplit - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
  }
  for (int idx = threadIdx.x; idx < nrows * R; idx += WARPS * 32) {
    const int r = idx / R, q = idx % R;
    float u = 0.f;
    if (ksplit > 1) {
      const float* part = a.partial + (size_t)item * ksplit * (MT * 16 * R) + idx;
      for (int k = 0; k < ksplit; ++k) u += __ldcg(part + (size_t)k * (MT * 16 * R));   // fixed order
    } else {
#pragma unroll
      for (int w = 0; w < WARPS; ++w) u += red[w][r][q];     // fixed order
    }
    const int row = rows[r];
    a.Out[(size_t)row * R + q] = u * sc;
    if (a.u_save && a.row_save) {
      const int sv = a.row_save[row];
      if (sv >= 0) a.u_save[(size_t)(a.save_base + sv) * R + q] = u;
    }
  }
  if (ksplit > 1 && threadIdx.x == 0) a.counters[item] = 0;     // ready for the next launch
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
__global__ void __launch_bounds__(GRAD_THREADS, MB == 1 ? 2 : 1)
grad_kernel(const GradArgs a) {
  extern __shared__ float grad_smem[];
  float (*red)[MB * 16][64 + 1] = reinterpret_cast<float (*)[MB * 16][64 + 1]>(grad_smem);
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
  // Two-deep register pipeline: the loads of chunk i+1 (4 rows of Q, 8 values of P per rank
  // block) are issued before the MMAs of chunk i.
  struct ChunkRegs { uint4 q[4]; float pv[MB][4][2]; };
  auto load_chunk = [&](int ch, ChunkRegs& r) {
    const int row0 = a.chunk_row0[ch], nrows = a.chunk_nrows[ch];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      r.q[i] = tr[i] < nrows ? ptx::ldg_nc_v4(a.Q + (size_t)(row0 + tr[i]) * a.ldq + j0 + 8 * g) : zero4;
#pragma unroll
    for (int m = 0; m < MB; ++m)
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int qq = qbase + m * 16 + g + 8 * h;      // pv[m][row index][q = g / g + 8]
          r.pv[m][i][h] = (tr[i] < nrows && qq < R) ? __ldg(a.P + (size_t)(row0 + tr[i]) * R + qq) : 0.f;
        }
  };
  constexpr int STEP = GRAD_THREADS / 32;
  ChunkRegs cur, nxt;
  int ch = ch0 + warp;
  if (ch < ch1) load_chunk(ch, cur);
  for (; ch < ch1; ch += STEP) {
    const bool more = ch + STEP < ch1;
    if (more) load_chunk(ch + STEP, nxt);
    uint32_t ahi[MB][4], alo[MB][4];
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      // fragment order: a0 (q=g, rows 2c,2c+1), a1 (q=g+8, rows 2c,2c+1), a2 (q=g, rows 2c+8,2c+9), a3
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const int h = f & 1, rp = (f >> 1) * 2;
        const float e0 = cur.pv[m][rp][h] * sc, e1 = cur.pv[m][rp + 1][h] * sc;
        const __nv_bfloat16 h0 = __float2bfloat16_rn(e0), h1 = __float2bfloat16_rn(e1);
        ahi[m][f] = ptx::pack_bf16(e0, e1);
        alo[m][f] = ptx::pack_bf16(e0 - __bfloat162float(h0), e1 - __bfloat162float(h1));
      }
    }
    const uint32_t qr[4][4] = {{cur.q[0].x, cur.q[0].y, cur.q[0].z, cur.q[0].w},
                               {cur.q[1].x, cur.q[1].y, cur.q[1].z, cur.q[1].w},
                               {cur.q[2].x, cur.q[2].y, cur.q[2].z, cur.q[2].w},
                               {cur.q[3].x, cur.q[3].y, cur.q[3].z, cur.q[3].w}};
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
    if (more) cur = nxt;
  }

  // every warp parks its accumulators; then all threads add the 8 partials in a fixed order.
  // column block nb, MMA column n  <->  strip column 8 n + nb
  {
    float (*mine)[64 + 1] = red[warp];
#pragma unroll
    for (int m = 0; m < MB; ++m)
#pragma unroll
      for (int nb = 0; nb < 8; ++nb) {
        const int ca = 8 * (2 * c) + nb, cb = 8 * (2 * c + 1) + nb;
        mine[m * 16 + g][ca] = acc[m][nb][0];
        mine[m * 16 + g][cb] = acc[m][nb][1];
        mine[m * 16 + g + 8][ca] = acc[m][nb][2];
        mine[m * 16 + g + 8][cb] = acc[m][nb][3];
      }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < MB * 16 * 64; idx += GRAD_THREADS) {
    const int ql = idx / 64, j = idx % 64;
    const int qq = qbase + ql;
    if (qq >= R) continue;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < GRAD_THREADS / 32; ++w) v += red[w][ql][j];
    float* dst = a.G + ((size_t)slot * R + qq) * a.D + j0 + j;
    *dst = a.accumulate ? (*dst + v) : v;
  }
}

}  // namespace mlora
