// Both LoRA gradients of a backward on the tcgen05 tensor cores, one launch:
//
//      dB_g = sum over the rows of slot g  (s u)^T dY          [r, d_out]      (problem 0)
//      dA_g = sum over the rows of slot g  V^T x               [r, d_in]       (problem 1; V from the shrink kernel)
//
// Both are G^T[cols, r] = Q^T P over the slot's rows: a tile of 128 rows of Q (dY or x_save; TMA, 128-byte
// swizzle) is read from shared memory as the MN-major A operand (M = 128 columns per MMA, K = the rows),
// P as the K-major N operand - bf16 head | remainder of the fp32 values (N = 2 r, about 16 mantissa bits;
// plain bf16 would leave errors of 2^-9 of the largest terms, which the tolerance on near-zero sums does
// not allow) - and the fp32 accumulators stay in tensor memory while the slot's row blocks stream by.  No register-file traffic for Q at all: the copy engine writes it, the
// tensor cores read it.
//
// Decomposition.  A slot's rows come as blocks of <= 128 rows (the plan's row blocks), the columns as
// strips of one tile width.  The tiles of both problems form one list, ordered problem > slot > strip > block,
// and every CTA of the persistent grid (one per SM) takes an equal contiguous range of it, so all SMs
// stream the same number of bytes whatever the shape.  The tiles of one (slot, strip) in a CTA's range
// form a PIECE.  With `snap` set (strips much shorter than a range) the ranges end at strip boundaries
// and every piece is whole; otherwise a piece that does not cover all blocks of its slot leaves its fp32
// sums in a per-CTA workspace and the CTA that arrives last at the strip's counter adds the pieces in
// CTA order (the order does not depend on who is last: run-to-run bit-reproducible).
//
// Warp roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer (also zeroes the rows of a short
// block's last 16-row step that belong to someone else), warps 2-5 convert P for up to NPB - 1 tiles
// ahead of the MMAs and drain finished pieces from tensor memory (two pieces' accumulators, so a drain
// overlaps the next piece's MMAs).  Piece counters are zero between launches: the CTA that leaves
// last clears them.  Every wait is bounded and reports through the status word.
#pragma once

#include <cuda.h>

#include "gemm_tcgen05.cuh"
#include "plan.h"
#include "ptx.cuh"

namespace mlora {
namespace gtc {

constexpr int ROWS = 128;                 // rows per tile (= the plan's row blocks)
constexpr int THREADS = 192;

__host__ __device__ constexpr uint32_t pow2_at_least(uint32_t x) {
  uint32_t p = 32;
  while (p < x) p *= 2;
  return p;
}

template <int R>
struct Cfg {
  static constexpr int N2 = 2 * R < 16 ? 16 : 2 * R;    // columns of one accumulator block: head | remainder of P
  static constexpr int CB = R <= 16 ? 4 : 2;            // 64-column blocks per tile
  static constexpr int S = R <= 16 ? 3 : (R <= 64 ? 5 : 3);    // stages of the tile ring (the copies in flight have to cover the memory latency)
  static constexpr int NPB = R <= 16 ? 4 : (R <= 32 ? 3 : 2);   // P operand buffers
  static constexpr int QC = R < 64 ? R : 64;            // rank rows drained from tensor memory at a time
  static constexpr int COLS = CB * 64;                  // tile (strip) width
  static constexpr uint32_t BLK = ROWS * 128;           // one 64-column block of a tile: [128 rows][128 B]
  static constexpr uint32_t STAGE_BYTES = CB * BLK;
  static constexpr uint32_t P_BYTES = 2 * N2 * 128;     // [2 K-blocks of 64 tile rows][N2 rows][128 B]
  static constexpr uint32_t ACC_COLS = (CB / 2) * N2;   // one piece's accumulators; two pieces in flight
  static constexpr uint32_t TMEM_COLS = pow2_at_least(2 * ACC_COLS);
  static constexpr uint32_t MISC_BYTES = 1024;
  static constexpr uint32_t SMEM_BYTES = 1024 + S * STAGE_BYTES + NPB * P_BYTES + MISC_BYTES;
  static constexpr int PIECE_FLOATS = R * COLS;         // fp32 sums one partial piece leaves behind
  static constexpr int F4 = PIECE_FLOATS / 4 / 128;     // float4 per thread of a piece
  static_assert(TMEM_COLS <= 512, "tensor memory");
  static_assert(SMEM_BYTES <= 232448, "shared memory");
};

struct Problem {
  const float* P;        // [T, R] fp32
  const float* scale;    // nullable: P multiplied by scale[slot's adapter]
  float* G;              // [n_slots, R, D]
  int32_t D, NS;         // columns, strips
};

struct Args {
  Problem prob[2];
  const int32_t* slot_adapter;   // [n_slots]
  const int32_t* slot_blk_off;   // [n_slots + 1]
  const int32_t* blk_row0;       // [NB] first compact row of the block
  const int32_t* blk_nrows;      // [NB]
  int32_t n_slots, NB;
  float* part_ws;                // [grid][4][PIECE_FLOATS] partial pieces: per problem, the piece a CTA's range opens with and the
                                 // one it closes with (a piece may still be waiting for its reader when its CTA has moved on)
  int32_t* counters;             // [n_counters]: [0] CTAs that have left, then one per (problem, slot, strip); zero between launches
  int32_t n_counters;
  int32_t accumulate;
  int32_t snap;                  // ranges end at strip boundaries (no partial pieces)
  int32_t* status;
  const uint8_t* pop;            // nullable: the P operands made ahead by psplit_kernel, [2 problems][NB][P_BYTES]
  const int32_t* slot_width;     // nullable (plans with per-adapter ranks, and only with pop): rank rows of a slot's gradient
                                 // that exist, w = 16 / 32 / 64 / 128; its operand image is then [2][2 w rows][128 B] (head | remainder
                                 // of w columns each), the MMAs have N = 2 w, and rows w .. R - 1 of the gradient are zero
};

// Position in one problem's tile list (slot > strip > block).
struct TileIt {
  const int32_t* off;    // slot_blk_off
  int NS, n_slots;
  int slot, strip, blk;  // blk: block index inside the slot
  int nb, b0;            // blocks of the slot, its first block
  __device__ __forceinline__ void seek(int t) {
    slot = 0;
    while (off[slot + 1] * NS <= t) ++slot;
    b0 = off[slot]; nb = off[slot + 1] - b0;
    const int rem = t - b0 * NS;
    strip = rem / nb;
    blk = rem - strip * nb;
  }
  __device__ __forceinline__ void next() {
    if (++blk < nb) return;
    blk = 0;
    if (++strip < NS) return;
    strip = 0;
    do { ++slot; } while (slot < n_slots - 1 && off[slot + 1] == off[slot]);
    if (slot >= n_slots) slot = n_slots - 1;               // past the end: never used
    b0 = off[slot]; nb = off[slot + 1] - b0;
  }
};

// The combined list holds N0 tiles of problem 0, then N1 of problem 1.  CTA c owns [begin(c), begin(c + 1)).
struct Ranges {
  int G, N0, N1, snap, n_slots;
  const int32_t* off;
  int NS0, NS1;
  __device__ __forceinline__ int begin(int c) const {
    const int N = N0 + N1;
    int g = (int)((long long)c * N / G);
    if (snap && g < N) {                                   // down to the first tile of the (slot, strip) it falls into
      const int p = g >= N0 ? 1 : 0;
      TileIt it{off, p ? NS1 : NS0, n_slots};
      it.seek(g - p * N0);
      g -= it.blk;
    }
    return g;
  }
  // this CTA's tiles of problem p, as indices into that problem's list
  __device__ __forceinline__ void of(int c, int p, int& t0, int& t1) const {
    const int lo = p ? N0 : 0, hi = p ? N0 + N1 : N0;
    const int g0 = begin(c), g1 = begin(c + 1);
    t0 = (g0 > lo ? g0 : lo) - lo;
    t1 = (g1 < hi ? g1 : hi) - lo;
  }
  // the CTA that owns tile t of problem p (plain ranges only: a snapped list has no shared strips)
  __device__ __forceinline__ int owner(int p, int t) const {
    const long long N = N0 + N1, g = (long long)t + (p ? N0 : 0);
    return (int)(((g + 1) * G + N - 1) / N) - 1;
  }
};

// The P operands of both problems, made once per block instead of once per tile: grid = (NB, 2, R / QC), 128
// threads, thread = row of the block, a CTA takes QC = 32 (rank 8, 16: all) of the low-rank columns.  Image of a block = what the kernel's operand buffer holds: (scaled) P[row, :] as
// bf16 head | remainder, [2 K-blocks of 64 rows][N2 columns][128 B] with the 16-byte pieces swizzled by the
// column index, rows past the block's end zero.  The gradient kernel then fetches an operand with one bulk copy.
__host__ __device__ constexpr int psplit_cols(int r) { return r < 32 ? r : 32; }

template <int R>
__global__ void __launch_bounds__(128)
psplit_kernel(const Args a, uint8_t* pop) {
  using C = Cfg<R>;
  constexpr int N2 = C::N2;
  const int blk = blockIdx.x, p = blockIdx.y, trow = threadIdx.x;
  const Problem& pr = a.prob[p];
  int slot = 0;
  while (slot + 1 < a.n_slots && a.slot_blk_off[slot + 1] <= blk) ++slot;
  const int nrows = a.blk_nrows[blk], row0 = a.blk_row0[blk];
  const bool live = trow < nrows;
  const float sc = pr.scale ? pr.scale[a.slot_adapter[slot]] : 1.0f;
  const int w = a.slot_width ? (a.slot_width[slot] < R ? a.slot_width[slot] : R) : R;     // columns that exist
  if ((int)blockIdx.z * psplit_cols(R) >= w) return;
  const int n2 = a.slot_width ? 2 * w : N2;                                                 // rows of a K-block of the image
  ptx::grid_dependency_wait();               // V comes from the launch before
  ptx::grid_launch_dependents();
  uint8_t* img = pop + ((size_t)p * a.NB + blk) * C::P_BYTES + (size_t)(trow >> 6) * ((uint32_t)n2 * 128u);
  const uint32_t kk = (uint32_t)(trow & 63);
  const float4* src = reinterpret_cast<const float4*>(pr.P + (size_t)(row0 + (live ? trow : 0)) * R);
  constexpr int QC = psplit_cols(R);
  {
    const int q0 = (int)blockIdx.z * QC;
    float pv[QC];
#pragma unroll
    for (int c0 = 0; c0 < QC; c0 += 4) {
      const float4 x = __ldg(src + ((q0 + c0) >> 2));
      pv[c0] = live ? x.x * sc : 0.f; pv[c0 + 1] = live ? x.y * sc : 0.f;
      pv[c0 + 2] = live ? x.z * sc : 0.f; pv[c0 + 3] = live ? x.w * sc : 0.f;
    }
#pragma unroll
    for (int c = 0; c < QC; ++c) {
      const int qq = q0 + c;
      if (qq >= w) break;                    // a narrower image ends here (its remainder rows start at w)
      const __nv_bfloat16 hi = __float2bfloat16_rn(pv[c]);
      const uint32_t off_hi = (uint32_t)qq * 128u + ((((kk >> 3) ^ (uint32_t)(qq & 7)) << 4) | ((kk & 7u) << 1));
      *reinterpret_cast<__nv_bfloat16*>(img + off_hi) = hi;
      const __nv_bfloat16 lo = __float2bfloat16_rn(pv[c] - __bfloat162float(hi));
      const uint32_t off_lo = (uint32_t)(w + qq) * 128u + ((((kk >> 3) ^ (uint32_t)((w + qq) & 7)) << 4) | ((kk & 7u) << 1));
      *reinterpret_cast<__nv_bfloat16*>(img + off_lo) = lo;
    }
  }
  if (2 * R < N2 && blockIdx.z == 0 && !a.slot_width) {       // (N2 = 2 R for every rank offered; kept for the layout's sake)
    for (int qq = 2 * R; qq < N2; ++qq)
      *reinterpret_cast<__nv_bfloat16*>(img + (uint32_t)qq * 128u + ((((kk >> 3) ^ (uint32_t)(qq & 7)) << 4) | ((kk & 7u) << 1))) =
          __float2bfloat16_rn(0.f);
  }
}

template <int R>
__global__ void __launch_bounds__(THREADS, 1)
grad_tc_kernel(const __grid_constant__ CUtensorMap tmQ0, const __grid_constant__ CUtensorMap tmQ1, const Args a) {
  using C = Cfg<R>;
  constexpr int CB = C::CB, NPB = C::NPB, N2 = C::N2, S = C::S;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_u32(smem_raw));
  auto s_stage = [&](int s) { return base + (uint32_t)s * C::STAGE_BYTES; };
  auto s_pbuf = [&](int b) { return base + S * C::STAGE_BYTES + (uint32_t)b * C::P_BYTES; };
  const uint32_t sBar = base + S * C::STAGE_BYTES + NPB * C::P_BYTES;
  // barriers: full[S] | empty[S] | pfull[NPB] | pempty[NPB] | accfull[2] | accempty[2] | esync
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (S + s); };
  auto bar_pfull = [&](int b) { return sBar + 8u * (2 * S + b); };
  auto bar_pempty = [&](int b) { return sBar + 8u * (2 * S + NPB + b); };
  auto bar_accfull = [&](int b) { return sBar + 8u * (2 * S + 2 * NPB + b); };
  auto bar_accempty = [&](int b) { return sBar + 8u * (2 * S + 2 * NPB + 2 + b); };
  const uint32_t bar_esync = sBar + 8u * (2 * S + 2 * NPB + 4);
  static_assert(8 * (2 * S + 2 * NPB + 5) <= 256, "barrier area");
  uint8_t* misc = gen + (sBar - base) + 256;
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 8);
  volatile int* last_flag = reinterpret_cast<volatile int*>(misc + 16);
  int* piece_off = reinterpret_cast<int*>(misc + 32);                      // [<= 160] workspace slots of the pieces being added up

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { ptx::mbar_init(bar_full(s), 1); ptx::mbar_init(bar_empty(s), 1); }
    for (int b = 0; b < NPB; ++b) { ptx::mbar_init(bar_pfull(b), 128); ptx::mbar_init(bar_pempty(b), 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(bar_accfull(b), 1); ptx::mbar_init(bar_accempty(b), 128); }
    ptx::mbar_init(bar_esync, 128);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ0);
    ptx::prefetch_tmap(&tmQ1);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  const Ranges rg{G, a.NB * a.prob[0].NS, a.NB * a.prob[1].NS, a.snap, a.n_slots, a.slot_blk_off, a.prob[0].NS, a.prob[1].NS};
  int rt0[2], rt1[2];                                       // this CTA's tiles of either problem (plan tables only)
  rg.of(cta, 0, rt0[0], rt1[0]);
  rg.of(cta, 1, rt0[1], rt1[1]);
  // only plan tables were read so far; the predecessor's outputs (V, and the counters it may still be
  // clearing) are touched after this point
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();

  if (warp == 0) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      uint32_t i = 0;
      bool ok = true;
      for (int p = 0; p < 2 && ok; ++p) {
        const int t0 = rt0[p], t1 = rt1[p];
        if (t0 >= t1) continue;
        TileIt it{a.slot_blk_off, a.prob[p].NS, a.n_slots};
        it.seek(t0);
        const CUtensorMap* tmQ = p ? &tmQ1 : &tmQ0;
        for (int t = t0; t < t1; ++t, ++i) {
          const int s = i % S;
          if (!(ok = gemm_wait(bar_empty(s), ((i / S) & 1) ^ 1, abort_flag, a.status))) break;
          ptx::mbar_arrive_expect_tx(bar_full(s), C::STAGE_BYTES);
          ptx::tma_load_3d(s_stage(s), tmQ, 0, a.blk_row0[it.b0 + it.blk], it.strip * CB, bar_full(s));
          if (t + 1 < t1) it.next();
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    uint32_t i = 0, n_piece = 0;
    bool ok = true;
    // the whole warp waits (one decision for all lanes); lane 0 issues
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, gemm_wait(bar, parity, abort_flag, a.status));
    };
    for (int p = 0; p < 2 && ok; ++p) {
      const int t0 = rt0[p], t1 = rt1[p];
      if (t0 >= t1) continue;
      TileIt it{a.slot_blk_off, a.prob[p].NS, a.n_slots};
      it.seek(t0);
      for (int t = t0; t < t1 && ok; ++t, ++i) {
        const int s = i % S, pb = i % NPB, ab = n_piece & 1;
        const bool first_piece = t == t0 || it.blk == 0, last_piece = t == t1 - 1 || it.blk == it.nb - 1;
        const int nrows = a.blk_nrows[it.b0 + it.blk];
        const int n2 = a.slot_width ? 2 * min(a.slot_width[it.slot], R) : N2;      // operand rows per K-block = the MMAs' N
        const uint32_t idesc = ptx::make_idesc_bf16(128, (uint32_t)n2, true, false);
        if (!(ok = wait_all(bar_pfull(pb), (i / NPB) & 1))) break;
        if (!(ok = wait_all(bar_full(s), (i / S) & 1))) break;
        const uint32_t q = s_stage(s);
        if (nrows & 15) {
          // rows of the block's last 16-row step that are not the block's own: they enter the gradient
          // multiplied by a zero of P, which would still spread a non-finite value - clear them
          const int r0 = nrows, nr = ((nrows + 15) & ~15) - nrows;
          for (int idx = lane; idx < nr * CB * 8; idx += 32) {
            const int pc = idx & 7, rr = r0 + (idx >> 3) % nr, cb = (idx >> 3) / nr;
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(q + (uint32_t)cb * C::BLK + (uint32_t)rr * 128u + (uint32_t)pc * 16u), "r"(0) : "memory");
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
        }
        if (first_piece && !(ok = wait_all(bar_accempty(ab), ((n_piece >> 1) & 1) ^ 1))) break;
        ptx::tc_fence_after();
        if (lane == 0) {
          const int ksteps = (nrows + 15) >> 4;
          const uint64_t bd0 = ptx::make_smem_desc(s_pbuf(pb), 16, 1024);
#pragma unroll
          for (int mb = 0; mb < CB / 2; ++mb) {
            const uint32_t d = tmem_base + (uint32_t)(ab * C::ACC_COLS + mb * N2);
            const uint64_t ad = ptx::make_smem_desc(q + (uint32_t)(2 * mb) * C::BLK, C::BLK, 1024);
            for (int ks = 0; ks < ksteps; ++ks)      // K-step ks: rows 16 ks .. of the tile; P's K-block ks / 4, 32 bytes per step inside it
              ptx::umma_f16(d, ad + (uint64_t)(ks * 128), bd0 + (uint64_t)((ks >> 2) * (n2 * 8) + (ks & 3) * 2), idesc,
                            (ks == 0 && first_piece) ? 0u : 1u);
          }
          ptx::umma_commit(bar_empty(s));
          ptx::umma_commit(bar_pempty(pb));
          if (last_piece) ptx::umma_commit(bar_accfull(ab));
        }
        __syncwarp();
        if (last_piece) ++n_piece;
        if (t + 1 < t1) it.next();
      }
    }
  } else {
    // ===================== operand conversion and piece drains (warps 2..5) =====================
    const int e = warp & 3;                    // the quarter of tensor memory this warp may read
    const int trow = e * 32 + lane;            // tile row this thread converts = accumulator lane it drains
    const uint32_t tlane = (uint32_t)(e * 32) << 16;
    const int tid = (int)threadIdx.x - 64;     // 0..127
    uint32_t ic = 0, n_piece = 0, n_sync = 0;  // tiles converted, pieces drained, meetings
    bool ok = true;

    // all four warps meet (bounded): an mbarrier rather than bar.sync, so that a warp that gave up cannot strand the others
    auto epi_sync = [&]() -> bool {
      ptx::mbar_arrive(bar_esync);
      const bool got = gemm_wait(bar_esync, n_sync & 1, abort_flag, a.status);
      ++n_sync;
      return __all_sync(0xffffffffu, got);
    };

    for (int p = 0; p < 2 && ok; ++p) {
      const Problem& pr = a.prob[p];
      const int t0 = rt0[p], t1 = rt1[p];
      if (t0 >= t1) continue;

      // ---- a tile's P operand: (scaled) P[row, :] as bf16 (head | remainder), K-major, 128-byte swizzle ----
      auto convert = [&](const TileIt& it) -> bool {
        const int blk_abs = it.b0 + it.blk;
        if (a.pop) {       // the operand image exists in memory: one bulk copy instead of a conversion per tile
          const int pb = ic % NPB;
          if (!__all_sync(0xffffffffu, gemm_wait(bar_pempty(pb), ((ic / NPB) & 1) ^ 1, abort_flag, a.status))) return false;
          if (tid == 0) {
            const uint32_t bytes = a.slot_width ? 512u * (uint32_t)min(a.slot_width[it.slot], R) : C::P_BYTES;   // [2][2 w][128 B]
            ptx::mbar_arrive_expect_tx(bar_pfull(pb), bytes);
            bulk_load(s_pbuf(pb), a.pop + ((size_t)p * a.NB + blk_abs) * C::P_BYTES, bytes, bar_pfull(pb));
          } else {
            ptx::mbar_arrive(bar_pfull(pb));
          }
          ++ic;
          return true;
        }
        const int nrows = a.blk_nrows[blk_abs], row0 = a.blk_row0[blk_abs];
        float pv[R];
        const bool live = trow < nrows;
        const float sc = pr.scale ? pr.scale[a.slot_adapter[it.slot]] : 1.0f;
        const float4* src = reinterpret_cast<const float4*>(pr.P + (size_t)(row0 + (live ? trow : 0)) * R);
#pragma unroll
        for (int c0 = 0; c0 < R; c0 += 4) {
          const float4 x = __ldg(src + (c0 >> 2));
          pv[c0] = live ? x.x * sc : 0.f; pv[c0 + 1] = live ? x.y * sc : 0.f;
          pv[c0 + 2] = live ? x.z * sc : 0.f; pv[c0 + 3] = live ? x.w * sc : 0.f;
        }
        const int pb = ic % NPB;
        if (!__all_sync(0xffffffffu, gemm_wait(bar_pempty(pb), ((ic / NPB) & 1) ^ 1, abort_flag, a.status))) return false;
        // element (n, k = tile row): K-block k / 64, row n of 128 bytes, 16-byte piece (k % 64) / 8 stored at piece ^ (n & 7)
        const uint32_t kb = s_pbuf(pb) + (uint32_t)(trow >> 6) * (N2 * 128u);
        const uint32_t kk = (uint32_t)(trow & 63);
#pragma unroll
        for (int qq = 0; qq < R; ++qq) {
          const __nv_bfloat16 hi = __float2bfloat16_rn(pv[qq]);
          const uint32_t off_hi = (uint32_t)qq * 128u + ((((kk >> 3) ^ (uint32_t)(qq & 7)) << 4) | ((kk & 7u) << 1));
          asm volatile("st.shared.b16 [%0], %1;" ::"r"(kb + off_hi), "h"(*reinterpret_cast<const uint16_t*>(&hi)) : "memory");
          const __nv_bfloat16 lo = __float2bfloat16_rn(pv[qq] - __bfloat162float(hi));
          const uint32_t off_lo = (uint32_t)(R + qq) * 128u + ((((kk >> 3) ^ (uint32_t)((R + qq) & 7)) << 4) | ((kk & 7u) << 1));
          asm volatile("st.shared.b16 [%0], %1;" ::"r"(kb + off_lo), "h"(*reinterpret_cast<const uint16_t*>(&lo)) : "memory");
        }
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(bar_pfull(pb));
        ++ic;
        return true;
      };

      TileIt itc{a.slot_blk_off, pr.NS, a.n_slots}, itd = itc;
      itc.seek(t0);
      itd.seek(t0);
      int tc = t0;                              // tiles [t0, tc) of this problem have their operand
      int piece_blk0 = 0;
      for (int t = t0; t < t1 && ok; ++t) {
        // operands for up to NPB - 1 tiles beyond this one: while a piece is being drained below, the MMAs go on
        while (ok && tc < t1 && tc < t + NPB) {
          if (tc > t0) itc.next();
          ok = convert(itc);
          ++tc;
        }
        if (!ok) break;
        const TileIt& it = itd;
        const bool first_piece = t == t0 || it.blk == 0, last_piece = t == t1 - 1 || it.blk == it.nb - 1;
        if (first_piece) piece_blk0 = it.blk;
        // ---- the piece's gradient sums, once its last tile is through ----
        if (last_piece) {
          const int ab = n_piece & 1;
          if (!(ok = __all_sync(0xffffffffu, gemm_wait(bar_accfull(ab), (n_piece >> 1) & 1, abort_flag, a.status)))) break;
          ptx::tc_fence_after();
          ++n_piece;
          const bool complete = piece_blk0 == 0 && it.blk == it.nb - 1;
          const int w = a.slot_width ? min(a.slot_width[it.slot], R) : R;  // rank rows that exist: head columns [0, w), remainder [w, 2 w)
          const int gbase = it.b0 * pr.NS + it.strip * it.nb;            // first tile of the (slot, strip)
          float* mine = a.part_ws + ((size_t)cta * 4 + p * 2 + (t0 >= gbase ? 0 : 1)) * C::PIECE_FLOATS;
#pragma unroll
          for (int mb = 0; mb < CB / 2; ++mb) {
            const int cl = mb * 128 + trow;                               // column inside the strip
            const int col = it.strip * C::COLS + cl;
            const uint32_t tacc = tmem_base + tlane + (uint32_t)(ab * C::ACC_COLS + mb * N2);
#pragma unroll
            for (int q0 = 0; q0 < R; q0 += C::QC) {                       // rank rows q0 .. q0 + QC: head columns and remainder columns
              uint32_t wh[C::QC < 16 ? 16 : C::QC], wl[C::QC < 16 ? 16 : C::QC];
#pragma unroll
              for (int c0 = 0; c0 < C::QC; c0 += 16) {
                if (q0 + c0 < w) {
                  ptx::tmem_ld_32x32b_x16(tacc + (uint32_t)(q0 + c0), wh + c0);
                  if (R >= 16) ptx::tmem_ld_32x32b_x16(tacc + (uint32_t)(w + q0 + c0), wl + c0);
                } else {                                                  // rows past the adapter's own rank: zero
#pragma unroll
                  for (int z = 0; z < 16; ++z) { wh[c0 + z] = 0u; wl[c0 + z] = 0u; }
                }
              }
              ptx::tmem_ld_wait();
              // rank 8: one load of 16 columns holds both halves
              auto val = [&](int qq) { return __uint_as_float(wh[qq]) + (R >= 16 ? __uint_as_float(wl[qq]) : __uint_as_float(wh[R + qq])); };
              if (complete) {
                if (col < pr.D) {
                  float* dst = pr.G + ((size_t)it.slot * R + q0) * pr.D + col;
                  if (a.accumulate) {
#pragma unroll
                    for (int qq = 0; qq < C::QC; ++qq) dst[(size_t)qq * pr.D] += val(qq);
                  } else {
#pragma unroll
                    for (int qq = 0; qq < C::QC; ++qq) dst[(size_t)qq * pr.D] = val(qq);
                  }
                }
              } else {
#pragma unroll
                for (int qq = 0; qq < C::QC; ++qq) mine[(q0 + qq) * C::COLS + cl] = val(qq);
              }
            }
          }
          ptx::tc_fence_before();
          ptx::mbar_arrive(bar_accempty(ab));
          if (!complete) {
            // ---- partial piece: the last CTA to arrive adds all pieces of the strip in CTA order ----
            __threadfence();
            const int c_first = rg.owner(p, gbase), c_last = rg.owner(p, gbase + it.nb - 1);
            const int lo = p ? rg.N0 : 0;
            // the pieces' workspace slots, in CTA order (a grid larger than the tile list leaves CTAs without tiles: no piece);
            for (int cc = c_first + tid; cc <= c_last; cc += 128) {
              const int g0 = rg.begin(cc), g1 = rg.begin(cc + 1);
              const int first_here = (g0 > lo ? g0 : lo) - lo;             // its first tile of this problem
              piece_off[cc - c_first] = g1 > g0 ? (cc * 4 + p * 2 + (first_here >= gbase ? 0 : 1)) : -1;
            }
            if (!(ok = epi_sync())) break;
            if (tid == 0) {
              int pieces = 0;
              for (int k = 0; k <= c_last - c_first; ++k) pieces += piece_off[k] >= 0 ? 1 : 0;
              int32_t* cnt = a.counters + 1 + (p ? a.n_slots * a.prob[0].NS : 0) + it.slot * pr.NS + it.strip;
              *last_flag = (atomicAdd(cnt, 1) == pieces - 1) ? 1 : 0;
            }
            if (!(ok = epi_sync())) break;
            if (*last_flag) {
              __threadfence();
              const int np = c_last - c_first + 1;
              float4 sum[C::F4];
#pragma unroll
              for (int k = 0; k < C::F4; ++k) sum[k] = make_float4(0.f, 0.f, 0.f, 0.f);
              for (int k2 = 0; k2 < np; ++k2) {
                const int slot_k = piece_off[k2];
                if (slot_k < 0) continue;
                const float4* src = reinterpret_cast<const float4*>(a.part_ws + (size_t)slot_k * C::PIECE_FLOATS) + tid;
#pragma unroll
                for (int k = 0; k < C::F4; ++k) {
                  const float4 x = __ldcg(src + k * 128);
                  sum[k].x += x.x; sum[k].y += x.y; sum[k].z += x.z; sum[k].w += x.w;
                }
              }
#pragma unroll
              for (int k = 0; k < C::F4; ++k) {
                const int f = k * 128 + tid;                                 // float4 index inside the piece: [qq][COLS / 4]
                const int qq = f / (C::COLS / 4), cl = (f - qq * (C::COLS / 4)) * 4;
                const int col = it.strip * C::COLS + cl;
                if (col >= pr.D) continue;
                float4* dst = reinterpret_cast<float4*>(pr.G + ((size_t)it.slot * R + qq) * pr.D + col);
                float4 o = sum[k];
                if (a.accumulate) { const float4 old = *dst; o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
                *dst = o;
              }
            }
            if (!(ok = epi_sync())) break;       // last_flag and piece_off are reused by the next piece
          }
        }
        if (t + 1 < t1) itd.next();
      }
    }
  }

  // ================================ common exit ================================
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
  // the CTA that leaves last puts every counter back to zero for the next launch
  if (threadIdx.x == 0) {
    __threadfence();
    *last_flag = (atomicAdd(a.counters, 1) == G - 1) ? 1 : 0;
  }
  __syncthreads();
  if (*last_flag) {
    for (int i = threadIdx.x; i < a.n_counters; i += THREADS) a.counters[i] = 0;
  }
}

}  // namespace gtc
}  // namespace mlora
