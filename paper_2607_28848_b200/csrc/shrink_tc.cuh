// The rank-r products U = X A_a^T (forward shrink) and V = s dY B_a^T (backward) on the tcgen05 tensor
// cores, for the higher ranks (the default from 32; at 64 and 128 the mma.sync kernels run out of registers and shared
// memory).
//
// Rows come as BLOCKS: runs of <= 128 consecutive rows that share one adapter (the plan's block tables).
// A block is one MMA operand: a tile of 128 rows x COLS columns of the input (TMA, 128-byte swizzle) is
// the K-major A operand (M = 128 rows, K = the columns), the adapter's r rows over the same columns the
// K-major N = r operand, and the [128, r] result accumulates in tensor memory while the block's column
// strips stream by.  Neither operand passes through registers.  Rows of the tile past the block's end
// belong to somebody else (or to nobody): they are multiplied and never read.
//
// Two launches.  shrink_tc_kernel: tiles ordered block > strip, every CTA of the persistent grid (one per
// SM) takes an equal contiguous range, the tiles of one block inside a range form a RUN with one
// accumulator (two in flight: a drain overlaps the next run's MMAs), and every run leaves its fp32 sums in
// a workspace, at rows [row0 + 128 cta, + nrows) - block index and CTA index both only grow along the
// tile order, so no two runs meet.  Nothing waits on another CTA.  shrink_tc_finish_kernel (programmatic
// dependent launch): 8 rows x r columns per CTA, adds a block's runs in CTA order (bit-reproducible),
// and writes what the step needs: the scaled fp32 result, the saved activations of fine-tuning rows (the
// unscaled result and a copy of the input rows), and the bf16 block-diagonal operand of the GEMM with its
// zeros.  A few hundred CTAs share the sums that one last-arriving CTA per block would otherwise do alone
// (19 runs of 64 KiB per block on a 14336-wide backward at rank 128).
//
// Every wait is bounded and reports through the status word.
#pragma once

#include <cuda.h>

#include "gemm_tcgen05.cuh"
#include "plan.h"
#include "ptx.cuh"
#include "skinny.cuh"

namespace mlora {
namespace stc {

constexpr int ROWS = 128;
constexpr int THREADS = 192;

template <int R>
struct Cfg {
  static constexpr int RP = R < 16 ? 16 : R;            // rank padded to the smallest N of a 128-row MMA
  static constexpr int CB = R <= 64 ? 4 : 2;            // 64-column blocks per tile
  static constexpr int S = R <= 16 ? 3 : (R <= 64 ? 2 : 3);   // stages (what fits 227 KiB)
  static constexpr int COLS = CB * 64;
  static constexpr uint32_t BLK = ROWS * 128;           // one 64-column block of a tile: [128 rows][128 B]
  static constexpr uint32_t Q_BYTES = CB * BLK;
  static constexpr uint32_t B_BYTES = CB * RP * 128;    // the adapter's rows over the tile's columns: [CB][RP rows][128 B]
  static constexpr uint32_t STAGE_BYTES = Q_BYTES + B_BYTES;
  static constexpr uint32_t TMEM_COLS = 2 * RP < 32 ? 32 : 2 * RP;
  static constexpr uint32_t SMEM_BYTES = 1024 + S * STAGE_BYTES + 1024;
  static constexpr int FIN_ROWS = R >= 16 ? 8 : 16;        // rows per CTA of the finish kernel (at least one full warp)
  static constexpr int FIN_THREADS = FIN_ROWS * (R / 4);   // one float4 of one row per thread
  static_assert(SMEM_BYTES <= 232448, "shared memory");
  static_assert(R % 8 == 0 && FIN_THREADS >= 32 && FIN_THREADS <= 1024, "finish kernel shape");
};

struct Args {
  const int32_t* blk_row0;       // [NB] first row of the block
  const int32_t* blk_nrows;      // [NB] 1 .. 128
  const int32_t* blk_adapter;    // [NB]
  const int32_t* blk_width;      // nullable (plans with per-adapter ranks): [NB] rows of the adapter's matrix the block needs, 16 / 32 / 64 / 128
  int32_t NB, NS;                // blocks, column strips per block
  float* part_ws;                // [rows + 128 * grid][R] fp32 sums of the runs
  int32_t* status;
};

struct FinArgs {
  const int32_t* blk_row0;
  const int32_t* blk_nrows;
  const int32_t* blk_adapter;
  const int32_t* blk_width;      // nullable: columns of the result that exist (the rest is written as zero)
  int32_t NB, NS, G;             // G: grid of the main kernel
  const float* part_ws;
  const float* scale;            // nullable: Out (and the operand chunks) multiplied by scale[adapter]
  float* Out;                    // [rows][R] fp32
  PbdArgs pbd;                   // bf16 block-diagonal copy for the GEMM (pbd.pbd may be null); pbd.scale applies on top
  // forward only (null / 0 otherwise): activation save of the fine-tuning rows
  const int32_t* row_save;       // [rows] save offset or -1
  float* u_save;                 // [cap][R]: the unscaled result
  const __nv_bfloat16* X;        // the input rows, row stride ldx
  int64_t ldx;
  __nv_bfloat16* x_save;         // [cap][D]
  int64_t save_base;
  int32_t D;
};

__host__ __device__ __forceinline__ int range_begin(int c, int G, int N) { return (int)((long long)c * N / G); }
__host__ __device__ __forceinline__ int owner(int t, int G, int N) { return (int)((((long long)t + 1) * G + N - 1) / N) - 1; }

template <int R>
__global__ void __launch_bounds__(THREADS, 1)
shrink_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmB16, const __grid_constant__ CUtensorMap tmB32,
                 const __grid_constant__ CUtensorMap tmB64, const Args a) {
  // tmB has boxes of RP rows (the whole padded adapter); tmB16 / 32 / 64 boxes of that many rows, for blocks whose
  // adapter has a smaller rank of its own (a.blk_width)
  using C = Cfg<R>;
  constexpr int RP = C::RP, CB = C::CB, S = C::S;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_u32(smem_raw));
  auto s_stage = [&](int s) { return base + (uint32_t)s * C::STAGE_BYTES; };
  const uint32_t sBar = base + S * C::STAGE_BYTES;
  // barriers: full[S] | empty[S] | vfull[2] | vempty[2]
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (S + s); };
  auto bar_vfull = [&](int v) { return sBar + 8u * (2 * S + v); };
  auto bar_vempty = [&](int v) { return sBar + 8u * (2 * S + 2 + v); };
  uint8_t* misc = gen + (sBar - base) + 128;
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  const int N = a.NB * a.NS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { ptx::mbar_init(bar_full(s), 1); ptx::mbar_init(bar_empty(s), 1); }
    for (int v = 0; v < 2; ++v) { ptx::mbar_init(bar_vfull(v), 1); ptx::mbar_init(bar_vempty(v), 128); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ);
    ptx::prefetch_tmap(&tmB);
    if (a.blk_width) { ptx::prefetch_tmap(&tmB16); ptx::prefetch_tmap(&tmB32); ptx::prefetch_tmap(&tmB64); }
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

  if (warp == 0) {
    // ================================ TMA producer ================================
    int blk = t0 < t1 ? t0 / a.NS : 0, strip = t0 - blk * a.NS;
    int row0 = 0, brow = 0, bw = RP;
    auto width_of = [&](int b) { const int w = a.blk_width ? a.blk_width[b] : RP; return w < RP ? w : RP; };
    if (t0 < t1) { row0 = a.blk_row0[blk]; brow = a.blk_adapter[blk] * R; bw = width_of(blk); }   // plan tables: readable before the wait
    ptx::grid_dependency_wait();             // the workspace may still be read by the launch before the last
    ptx::grid_launch_dependents();
    if (lane == 0) {
      bool ok = true;
      for (int t = t0, i = 0; t < t1 && ok; ++t, ++i) {
        const int s = i % S;
        if (!(ok = gemm_wait(bar_empty(s), ((i / S) & 1) ^ 1, abort_flag, a.status))) break;
        ptx::mbar_arrive_expect_tx(bar_full(s), C::Q_BYTES + (uint32_t)(CB * bw * 128));
        ptx::tma_load_3d(s_stage(s), &tmQ, 0, row0, strip * CB, bar_full(s));
        // the adapter's rows over the tile's columns: [CB][bw rows][128 B]
        const CUtensorMap* mb = bw >= RP ? &tmB : (bw == 16 ? &tmB16 : (bw == 32 ? &tmB32 : &tmB64));
        ptx::tma_load_3d(s_stage(s) + C::Q_BYTES, mb, 0, brow, strip * CB, bar_full(s));
        if (++strip == a.NS && t + 1 < t1) {
          strip = 0; ++blk;
          row0 = a.blk_row0[blk]; brow = a.blk_adapter[blk] * R; bw = width_of(blk);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    if (lane == 0) {
      uint32_t n_run = 0;
      bool ok = true;
      int cur_blk = -1, bw = RP;
      uint32_t idesc = ptx::make_idesc_bf16(128, RP, false, false);
      for (int t = t0, i = 0; t < t1 && ok; ++t, ++i) {
        const int s = i % S, blk = t / a.NS, strip = t - blk * a.NS;
        if (blk != cur_blk) {                  // N = the rows of the adapter's matrix this block reads
          cur_blk = blk;
          const int w = a.blk_width ? a.blk_width[blk] : RP;
          bw = w < RP ? w : RP;
          idesc = ptx::make_idesc_bf16(128, (uint32_t)bw, false, false);
        }
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
          const uint64_t bd = ptx::make_smem_desc(q + C::Q_BYTES + (uint32_t)cb * ((uint32_t)bw * 128u), 16, 1024);
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
    uint32_t n_run = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int blk = t / a.NS, strip0 = t - blk * a.NS;
      const int len = min(a.NS - strip0, t1 - t);           // this run: strips strip0 .. strip0 + len of the block
      const int nrows = a.blk_nrows[blk];
      const int bwid = a.blk_width ? min(a.blk_width[blk], RP) : RP;       // columns that exist (the same for the whole warp)
      float* dst = a.part_ws + ((size_t)a.blk_row0[blk] + (size_t)128 * cta + trow) * R;
      const int v = n_run & 1;
      if (!(ok = __all_sync(0xffffffffu, gemm_wait(bar_vfull(v), (n_run >> 1) & 1, abort_flag, a.status)))) break;
      ptx::tc_fence_after();
      ++n_run;
      constexpr int QC = R < 64 ? (R < 16 ? 16 : R) : 64;   // columns per round of loads
#pragma unroll
      for (int q0 = 0; q0 < RP; q0 += QC) {
        if (q0 >= bwid) break;
        uint32_t vv[QC];
#pragma unroll
        for (int c0 = 0; c0 < QC; c0 += 16) ptx::tmem_ld_32x32b_x16(tmem_base + tlane + (uint32_t)(v * RP + q0 + c0), vv + c0);
        ptx::tmem_ld_wait();
        if (trow < nrows) {
#pragma unroll
          for (int c0 = 0; c0 < QC; c0 += 4)
            if (q0 + c0 < R && q0 + c0 < bwid)
              *reinterpret_cast<float4*>(dst + q0 + c0) = make_float4(__uint_as_float(vv[c0]), __uint_as_float(vv[c0 + 1]),
                                                                      __uint_as_float(vv[c0 + 2]), __uint_as_float(vv[c0 + 3]));
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_vempty(v));
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
}

// grid = (NB + ceil(n_zero_rows / FIN_ROWS), 128 / FIN_ROWS), FIN_ROWS * R / 4 threads: thread (r, j) owns
// columns 4j .. 4j+3 of row r of its FIN_ROWS rows of a block.
template <int R>
__global__ void __launch_bounds__(Cfg<R>::FIN_THREADS)
shrink_tc_finish_kernel(const FinArgs a) {
  constexpr int TPR = R / 4;                 // threads per row
  constexpr int FIN_ROWS = Cfg<R>::FIN_ROWS;
  const int r_in = (int)threadIdx.x / TPR, j = (int)threadIdx.x % TPR;
  if ((int)blockIdx.x >= a.NB) {
    // ---- rows without an adapter inside tiles that have groups: all-zero operand chunks ----
    if (blockIdx.y != 0 || !a.pbd.pbd) return;
    const int zi = ((int)blockIdx.x - a.NB) * FIN_ROWS + r_in;
    if (zi >= a.pbd.n_zero_rows) return;
    const int row = a.pbd.zero_rows[zi];
    const int tile = row >> 8, rl = row & 255;
    const int goff = a.pbd.tile2_grp_off[tile], Gt = a.pbd.tile2_grp_off[tile + 1] - goff;
    const int LC = ((a.pbd.tile2_cols ? a.pbd.tile2_cols[tile] : Gt * R) + 63) / 64;
    __nv_bfloat16* base = a.pbd.pbd + ((size_t)(2 * goff) * 256 + rl) * 64;
    for (int pi = j; pi < LC * 8; pi += TPR)
      *reinterpret_cast<uint4*>(base + (size_t)(pi >> 3) * (256 * 64) + (pi & 7) * 8) = make_uint4(0, 0, 0, 0);
    return;
  }
  const int blk = blockIdx.x;
  const int nrows = a.blk_nrows[blk];
  if ((int)blockIdx.y * FIN_ROWS >= nrows) return;
  const int r = (int)blockIdx.y * FIN_ROWS + r_in;
  const bool live = r < nrows;
  const bool exists = !a.blk_width || 4 * j < a.blk_width[blk];     // columns past the adapter's own rank: zero, nothing to add
  const int row0 = a.blk_row0[blk], row = row0 + (live ? r : 0);
  const int ad = a.blk_adapter[blk];
  const float sc = a.scale ? a.scale[ad] : 1.0f;
  const float psc = a.pbd.scale ? a.pbd.scale[ad] : 1.0f;
  const int sv = (live && a.row_save) ? a.row_save[row] : -1;
  int goff = 0, g = -1, cols = 0, c0 = 0, cw = 0;     // the tile's operand columns; the row's own: [c0, c0 + cw)
  if (a.pbd.pbd) {
    const int tile = row >> 8;
    goff = a.pbd.tile2_grp_off[tile];
    g = a.pbd.row_grp2[row];
    cols = a.pbd.tile2_cols ? a.pbd.tile2_cols[tile] : (a.pbd.tile2_grp_off[tile + 1] - goff) * R;
    if (g >= 0) {
      c0 = a.pbd.grp2_col ? a.pbd.grp2_col[goff + g] : g * R;
      cw = a.pbd.grp2_width ? a.pbd.grp2_width[goff + g] : R;
    }
  }
  const int N = a.NB * a.NS, gbase = blk * a.NS;
  const int c_first = owner(gbase, a.G, N), c_last = owner(gbase + a.NS - 1, a.G, N);
  // the copy of the input rows needs nothing of the main kernel: do it before the wait
  if (sv >= 0 && a.x_save) {
    const uint4* src = reinterpret_cast<const uint4*>(a.X + (size_t)row * a.ldx);
    uint4* dst = reinterpret_cast<uint4*>(a.x_save + (size_t)(a.save_base + sv) * a.D);
    for (int k = j; k < a.D / 8; k += TPR) dst[k] = __ldg(src + k);
  }
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
  {
    const float* src = a.part_ws + ((size_t)row0 + r) * R + 4 * j;
    // runs in CTA order, eight loads in flight (the main grid never has more CTAs than tiles, so every CTA
    // from c_first to c_last has tiles of this block)
    for (int c0 = c_first; c0 <= c_last; c0 += 8) {
      float4 x[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int cc = c0 + k;
        x[k] = (live && exists && cc <= c_last) ? __ldcg(reinterpret_cast<const float4*>(src + (size_t)128 * cc * R))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) { sum.x += x[k].x; sum.y += x[k].y; sum.z += x[k].z; sum.w += x[k].w; }
    }
  }
  const float4 vs = make_float4(sum.x * sc, sum.y * sc, sum.z * sc, sum.w * sc);
  if (live) {
    *reinterpret_cast<float4*>(a.Out + (size_t)row * R + 4 * j) = vs;
    if (sv >= 0 && a.u_save) *reinterpret_cast<float4*>(a.u_save + (size_t)(a.save_base + sv) * R + 4 * j) = sum;
  }
  if (a.pbd.pbd) {
    // the row's chunks of the block-diagonal operand: thread pairs (2i, 2i + 1) hold one 16-byte piece
    uint32_t w0 = ptx::pack_bf16(vs.x * psc, vs.y * psc), w1 = ptx::pack_bf16(vs.z * psc, vs.w * psc);
    const uint32_t n0 = __shfl_down_sync(0xffffffffu, w0, 1), n1 = __shfl_down_sync(0xffffffffu, w1, 1);
    if (live) {
      const int LC = (cols + 63) / 64;
      __nv_bfloat16* base = a.pbd.pbd + ((size_t)(2 * goff) * 256 + (row & 255)) * 64;
      const int p0 = g >= 0 ? c0 / 8 : LC * 8, pw = cw / 8;     // the row's own 16-byte pieces: [p0, p0 + pw)
      if (g >= 0 && (j & 1) == 0 && (j >> 1) < pw) {
        const int pi = p0 + (j >> 1);
        *reinterpret_cast<uint4*>(base + (size_t)(pi >> 3) * (256 * 64) + (pi & 7) * 8) = make_uint4(w0, w1, n0, n1);
      }
      for (int pi = j; pi < LC * 8; pi += TPR)
        if (pi < p0 || pi >= p0 + pw)
          *reinterpret_cast<uint4*>(base + (size_t)(pi >> 3) * (256 * 64) + (pi & 7) * 8) = make_uint4(0, 0, 0, 0);
    }
  }
}

}  // namespace stc
}  // namespace mlora
