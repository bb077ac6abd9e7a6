// V = s dY B_a^T for the fine-tuning rows of a backward, on the tcgen05 tensor cores.
//
// The compact fine-tuning rows come as blocks of <= 128 rows that share one adapter (the plan's row
// blocks), so a block is one MMA operand: a tile of 128 rows x COLS columns of dY (TMA, 128-byte swizzle)
// is the K-major A operand (M = 128 rows, K = the columns), the adapter's rows of B over the same columns
// the K-major N = r operand, and V[128, r] accumulates in tensor memory while the block's column strips
// stream by.  Neither operand passes through registers.
//
// Decomposition.  Tiles are ordered block > strip and every CTA of the persistent grid (one per SM) takes
// an equal contiguous range, so all SMs stream the same number of bytes.  The tiles of one block in a
// CTA's range form a RUN with one accumulator (two runs in flight: a drain overlaps the next run's MMAs).
// A run that covers all strips of its block finishes it: scale, fp32 V for the gradient kernel, bf16
// block-diagonal chunks for the input-gradient GEMM.  Otherwise it leaves its fp32 sums in a per-CTA
// workspace and the CTA that arrives last at the block's counter adds the runs in CTA order (the order
// does not depend on who is last: run-to-run bit-reproducible) and finishes the block.  Nothing waits on
// another CTA.  Counters are zero between launches: the CTA that leaves last clears them.  Every wait is
// bounded and reports through the status word.
//
// Warp roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 drains (thread = row).
#pragma once

#include <cuda.h>

#include "gemm_tcgen05.cuh"
#include "plan.h"
#include "ptx.cuh"
#include "skinny.cuh"

namespace mlora {
namespace vtc {

constexpr int ROWS = 128;
constexpr int THREADS = 192;

template <int R>
struct Cfg {
  static constexpr int RP = R < 16 ? 16 : R;            // rank padded to the smallest N of a 128-row MMA
  static constexpr int CB = R <= 16 ? 4 : 2;            // 64-column blocks per tile
  static constexpr int S = R <= 16 ? 3 : (R == 32 ? 5 : (R == 64 ? 4 : 3));   // stages
  static constexpr int COLS = CB * 64;
  static constexpr uint32_t BLK = ROWS * 128;           // one 64-column block of a tile: [128 rows][128 B]
  static constexpr uint32_t Q_BYTES = CB * BLK;
  static constexpr uint32_t B_BYTES = CB * RP * 128;    // the adapter's rows over the tile's columns: [CB][RP rows][128 B]
  static constexpr uint32_t STAGE_BYTES = Q_BYTES + B_BYTES;
  static constexpr uint32_t TMEM_COLS = 2 * RP < 32 ? 32 : 2 * RP;
  static constexpr uint32_t SMEM_BYTES = 1024 + S * STAGE_BYTES + 1024;
  static constexpr int RUN_FLOATS = ROWS * R;           // fp32 sums one partial run leaves behind: [row][R]
  static_assert(SMEM_BYTES <= 232448, "shared memory");
  static_assert(RUN_FLOATS * 4 <= 65536, "a run's sums fit one workspace slot");
};

struct Args {
  const float* scale;            // [n_adapters]
  const int32_t* blk_row0;       // [NB] first compact row of the block
  const int32_t* blk_nrows;      // [NB]
  const int32_t* row_adapter;    // [T] adapter of a compact row (a block's rows share it)
  int32_t NB, NS, D;
  float* V_out;                  // [T, R] fp32, scaled
  PbdArgs pbd;                   // bf16 block-diagonal copy for the GEMM (pbd.pbd may be null)
  float* part_ws;                // [grid][4][16384 floats]: slot 0 the run a CTA's range opens with, slot 1 the one it closes with
  int32_t* counters;             // [1 + NB]: [0] CTAs that have left, then one per block; zero between launches
  int32_t* status;
};

__device__ __forceinline__ int range_begin(int c, int G, int N) { return (int)((long long)c * N / G); }
__device__ __forceinline__ int owner(int t, int G, int N) { return (int)((((long long)t + 1) * G + N - 1) / N) - 1; }

// One thread writes all chunks of its row of the block-diagonal operand (see PbdArgs): 16-byte pieces, the
// row's own group block carries bf16(vals), everything else zero.
template <int R>
__device__ __forceinline__ void pbd_write_row_thread(const PbdArgs& pa, int row, const float* vals) {
  const int tile = row >> 8, rl = row & 255;
  const int goff = pa.tile2_grp_off[tile], G = pa.tile2_grp_off[tile + 1] - goff, g = pa.row_grp2[row];
  const int LC = (G * R + 63) / 64;
  __nv_bfloat16* base = pa.pbd + ((size_t)(2 * goff) * 256 + rl) * 64;     // chunk c of the row: base + c * 256 * 64
  const int p0 = g >= 0 ? g * (R / 8) : LC * 8;          // the row's own pieces: p0 .. p0 + R / 8 (a piece = 8 low-rank columns)
  for (int pi = 0; pi < LC * 8; ++pi)                    // everything outside them is zero
    if (pi < p0 || pi >= p0 + R / 8)
      *reinterpret_cast<uint4*>(base + (size_t)(pi >> 3) * (256 * 64) + (pi & 7) * 8) = make_uint4(0, 0, 0, 0);
  if (g >= 0) {
#pragma unroll
    for (int j = 0; j < R / 8; ++j) {
      const int pi = p0 + j;
      uint4 v;
      v.x = ptx::pack_bf16(vals[8 * j], vals[8 * j + 1]); v.y = ptx::pack_bf16(vals[8 * j + 2], vals[8 * j + 3]);
      v.z = ptx::pack_bf16(vals[8 * j + 4], vals[8 * j + 5]); v.w = ptx::pack_bf16(vals[8 * j + 6], vals[8 * j + 7]);
      *reinterpret_cast<uint4*>(base + (size_t)(pi >> 3) * (256 * 64) + (pi & 7) * 8) = v;
    }
  }
}

template <int R>
__global__ void __launch_bounds__(THREADS, 1)
vshrink_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmB, const Args a) {
  using C = Cfg<R>;
  constexpr int RP = C::RP, CB = C::CB, S = C::S;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_u32(smem_raw));
  auto s_stage = [&](int s) { return base + (uint32_t)s * C::STAGE_BYTES; };
  const uint32_t sBar = base + S * C::STAGE_BYTES;
  // barriers: full[S] | empty[S] | vfull[2] | vempty[2] | esync
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (S + s); };
  auto bar_vfull = [&](int v) { return sBar + 8u * (2 * S + v); };
  auto bar_vempty = [&](int v) { return sBar + 8u * (2 * S + 2 + v); };
  const uint32_t bar_esync = sBar + 8u * (2 * S + 4);
  uint8_t* misc = gen + (sBar - base) + 128;
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 8);
  volatile int* last_flag = reinterpret_cast<volatile int*>(misc + 16);
  int* piece_off = reinterpret_cast<int*>(misc + 32);                      // [<= 160] workspace slots of the runs being added up

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  const int N = a.NB * a.NS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { ptx::mbar_init(bar_full(s), 1); ptx::mbar_init(bar_empty(s), 1); }
    for (int v = 0; v < 2; ++v) { ptx::mbar_init(bar_vfull(v), 1); ptx::mbar_init(bar_vempty(v), 128); }
    ptx::mbar_init(bar_esync, 128);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  const int t0 = range_begin(cta, G, N), t1 = range_begin(cta + 1, G, N);
  // only plan tables were read so far; the predecessor's outputs are touched after this point
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();

  if (warp == 0) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      bool ok = true;
      for (int t = t0, i = 0; t < t1 && ok; ++t, ++i) {
        const int s = i % S, blk = t / a.NS, strip = t - blk * a.NS;
        if (!(ok = gemm_wait(bar_empty(s), ((i / S) & 1) ^ 1, abort_flag, a.status))) break;
        const int row0 = a.blk_row0[blk];
        ptx::mbar_arrive_expect_tx(bar_full(s), C::STAGE_BYTES);
        ptx::tma_load_3d(s_stage(s), &tmQ, 0, row0, strip * CB, bar_full(s));
        ptx::tma_load_3d(s_stage(s) + C::Q_BYTES, &tmB, 0, a.row_adapter[row0] * R, strip * CB, bar_full(s));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(128, RP, false, false);
      uint32_t n_run = 0;
      bool ok = true;
      for (int t = t0, i = 0; t < t1 && ok; ++t, ++i) {
        const int s = i % S, blk = t / a.NS, strip = t - blk * a.NS;
        const bool first = t == t0 || strip == 0, last = t == t1 - 1 || strip == a.NS - 1;
        const int v = n_run & 1;
        if (first && !(ok = gemm_wait(bar_vempty(v), ((n_run >> 1) & 1) ^ 1, abort_flag, a.status))) break;
        if (!(ok = gemm_wait(bar_full(s), (i / S) & 1, abort_flag, a.status))) break;
        ptx::tc_fence_after();
        const uint32_t q = s_stage(s), d = tmem_base + (uint32_t)(v * RP);
        uint32_t acc = first ? 0u : 1u;
#pragma unroll
        for (int cb = 0; cb < CB; ++cb) {
          const uint64_t ad = ptx::make_smem_desc(q + (uint32_t)cb * C::BLK, 16, 1024);
          const uint64_t bd = ptx::make_smem_desc(q + C::Q_BYTES + (uint32_t)cb * (RP * 128u), 16, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            ptx::umma_f16(d, ad + (uint64_t)(ks * 2), bd + (uint64_t)(ks * 2), idesc, acc);
            acc = 1;
          }
        }
        ptx::umma_commit(bar_empty(s));
        if (last) { ptx::umma_commit(bar_vfull(v)); ++n_run; }
      }
    }
    __syncwarp();
  } else {
    // ================================ drains (warps 2..5, thread = row) ================================
    const int e = warp & 3;
    const int trow = e * 32 + lane;
    const uint32_t tlane = (uint32_t)(e * 32) << 16;
    const int tid = (int)threadIdx.x - 64;
    uint32_t n_run = 0, n_sync = 0;
    bool ok = true;
    auto epi_sync = [&]() -> bool {
      ptx::mbar_arrive(bar_esync);
      const bool got = gemm_wait(bar_esync, n_sync & 1, abort_flag, a.status);
      ++n_sync;
      return __all_sync(0xffffffffu, got);
    };
    // a finished block's rows: scale, fp32 for the gradient kernel, bf16 chunks for the GEMM
    auto finish_row = [&](int blk, float* vals) {
      const int nrows = a.blk_nrows[blk], row = a.blk_row0[blk] + trow;
      if (trow >= nrows) return;
      const float sc = a.scale[a.row_adapter[row]];
#pragma unroll
      for (int qq = 0; qq < R; ++qq) vals[qq] *= sc;
      float4* dst = reinterpret_cast<float4*>(a.V_out + (size_t)row * R);
#pragma unroll
      for (int c0 = 0; c0 < R; c0 += 4) dst[c0 >> 2] = make_float4(vals[c0], vals[c0 + 1], vals[c0 + 2], vals[c0 + 3]);
      if (a.pbd.pbd) pbd_write_row_thread<R>(a.pbd, row, vals);
    };
    for (int t = t0; t < t1 && ok;) {
      const int blk = t / a.NS, strip0 = t - blk * a.NS;
      const int len = min(a.NS - strip0, t1 - t);           // this run: strips strip0 .. strip0 + len of the block
      const int v = n_run & 1;
      if (!(ok = __all_sync(0xffffffffu, gemm_wait(bar_vfull(v), (n_run >> 1) & 1, abort_flag, a.status)))) break;
      ptx::tc_fence_after();
      ++n_run;
      uint32_t vv[RP];
#pragma unroll
      for (int c0 = 0; c0 < RP; c0 += 16) ptx::tmem_ld_32x32b_x16(tmem_base + tlane + (uint32_t)(v * RP + c0), vv + c0);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_vempty(v));
      float* vals = reinterpret_cast<float*>(vv);
      if (len == a.NS) {
        finish_row(blk, vals);
      } else {
        // ---- the block is shared with other CTAs: leave the sums, the last one to arrive adds them in CTA order ----
        const int gbase = blk * a.NS;
        float4* mine = reinterpret_cast<float4*>(a.part_ws + ((size_t)cta * 4 + (t0 >= gbase ? 0 : 1)) * 16384 + (size_t)trow * R);
#pragma unroll
        for (int c0 = 0; c0 < R; c0 += 4) mine[c0 >> 2] = make_float4(vals[c0], vals[c0 + 1], vals[c0 + 2], vals[c0 + 3]);
        __threadfence();
        const int c_first = owner(gbase, G, N), c_last = owner(gbase + a.NS - 1, G, N);
        for (int cc = c_first + tid; cc <= c_last; cc += 128) {
          const int rb = range_begin(cc, G, N);
          piece_off[cc - c_first] = range_begin(cc + 1, G, N) > rb ? (cc * 4 + (rb >= gbase ? 0 : 1)) : -1;
        }
        if (!(ok = epi_sync())) break;
        if (tid == 0) {
          int pieces = 0;
          for (int k = 0; k <= c_last - c_first; ++k) pieces += piece_off[k] >= 0 ? 1 : 0;
          *last_flag = (atomicAdd(a.counters + 1 + blk, 1) == pieces - 1) ? 1 : 0;
        }
        if (!(ok = epi_sync())) break;
        if (*last_flag) {
          __threadfence();
          float sum[R];
#pragma unroll
          for (int qq = 0; qq < R; ++qq) sum[qq] = 0.f;
          // the runs are added in CTA order; their loads go out KB runs at a time (one round trip to the L2 per batch)
          constexpr int KB = R <= 16 ? 4 : (R <= 32 ? 2 : 1);
          const int np = c_last - c_first + 1;
          for (int k0 = 0; k0 < np; k0 += KB) {
            float4 x[KB][R / 4];
#pragma unroll
            for (int kk = 0; kk < KB; ++kk) {
              const int slot_k = k0 + kk < np ? piece_off[k0 + kk] : -1;
              const float4* src = reinterpret_cast<const float4*>(a.part_ws + (size_t)(slot_k < 0 ? 0 : slot_k) * 16384 + (size_t)trow * R);
#pragma unroll
              for (int c = 0; c < R / 4; ++c) x[kk][c] = slot_k < 0 ? make_float4(0.f, 0.f, 0.f, 0.f) : __ldcg(src + c);
            }
#pragma unroll
            for (int kk = 0; kk < KB; ++kk)
#pragma unroll
              for (int c = 0; c < R / 4; ++c) {
                sum[4 * c] += x[kk][c].x; sum[4 * c + 1] += x[kk][c].y; sum[4 * c + 2] += x[kk][c].z; sum[4 * c + 3] += x[kk][c].w;
              }
          }
          finish_row(blk, sum);
        }
        if (!(ok = epi_sync())) break;        // last_flag and piece_off are reused by the next run
      }
      t += len;
    }
  }

  // ================================ common exit ================================
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
  if (threadIdx.x == 0) {
    __threadfence();
    *last_flag = (atomicAdd(a.counters, 1) == G - 1) ? 1 : 0;
  }
  __syncthreads();
  if (*last_flag) {
    for (int i = threadIdx.x; i <= a.NB; i += THREADS) a.counters[i] = 0;
  }
}

}  // namespace vtc
}  // namespace mlora
