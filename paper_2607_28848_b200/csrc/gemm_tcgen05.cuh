// Tensor-core kernel of the mixed-batch multi-LoRA layer:
//
//      Out[m, :] = In[m, :] * Wop  +  P[m, :] * L_{a(m)}
//
// with In [M, K] (bf16, K contiguous), Wop the frozen base weight (either [K, N] with N
// contiguous, the forward, or [N, K] with K contiguous, the input-gradient pass), P [M, R] the
// rank-R intermediate of each row (fp32, optionally multiplied by the adapter's scale) and
// L_a [R, N] the adapter's expand matrix (N contiguous).  Forward: In = X, L = B, P = X A^T.
// Input gradient: In = dY, Wop = W read transposed, L = A, P = V = s dY B^T.
//
// One persistent CTA per SM walks 128 x 256 output tiles.  Per tile the contraction runs over
// K in blocks of 64 (TMA -> 128B-swizzled shared memory -> tcgen05.mma into a 128 x 256 fp32
// accumulator in tensor memory) and is then EXTENDED by the low-rank part: the rows' P values
// are laid out block-diagonally by adapter ("groups" of the tile) as an extra A operand, the
// groups' L_a tiles are stacked as the matching B operand, and a few more tcgen05.mma steps add
// s (x A^T) B into the same accumulator.  The output tile is therefore written exactly once.
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer (owns tensor memory),
// warps 2-5 epilogue (tensor memory -> registers -> bf16 -> shared -> TMA store), warps 6-9
// build the low-rank A operand in shared memory.  Two accumulators (2 x 256 columns) let the
// epilogue of one tile overlap the main loop of the next.
//
// Every wait is bounded: when one runs out the CTA raises a shared abort flag, records
// MLORA_ERR_DEVICE_TIMEOUT in the status word, and all roles fall through to the common exit
// where tensor memory is released.
#pragma once

#include <cuda.h>

#include "ptx.cuh"

namespace mlora {

constexpr int GEMM_BM = 128;
constexpr int GEMM_BN = 256;
constexpr int GEMM_BK = 64;
constexpr int GEMM_STAGES = 4;
constexpr int GEMM_THREADS = 320;
constexpr uint32_t GEMM_A_BYTES = GEMM_BM * GEMM_BK * 2;             // 16 KiB
constexpr uint32_t GEMM_B_BYTES = GEMM_BN * GEMM_BK * 2;             // 32 KiB
constexpr uint32_t GEMM_STAGE_BYTES = GEMM_A_BYTES + GEMM_B_BYTES;   // 48 KiB
constexpr uint32_t GEMM_EPI_BYTES = 4 * 2 * 4096;                    // 4 warps x 2 buffers x (32 rows x 128 B)
constexpr uint32_t GEMM_SMEM_BYTES = GEMM_STAGES * GEMM_STAGE_BYTES + GEMM_EPI_BYTES + 256 + 1024;
constexpr uint32_t GEMM_SPIN_LIMIT = 1u << 22;
constexpr uint32_t GEMM_TMEM_COLS = 512;

struct GemmArgs {
  int32_t M, N, K;
  int32_t n_mtiles, n_ntiles;
  int32_t n_full;                // work units [0, n_full) are whole 128 x 256 tiles; the tiles after
  int32_t n_units;               // them (the last, partly filled wave) are cut into two 128 x 128 halves
  int32_t lora_enabled;
  int32_t group_m;               // two-SM kernel only: row tiles per band of the tile order (0: one band)
  // Two-SM kernel only: tiles [0, n_whole) are whole work units; each of the n_tail tiles after them is
  // cut into split_k K slices (units after the whole ones, slice-major), whose fp32 partial tiles go
  // to ws_splitk[slice][tail tile][256][256] and are added up by splitk_reduce_kernel.  n_tail = 0:
  // no split; n_whole = 0: every tile is split (few tiles for the SMs); otherwise only the tiles of
  // the last, partly filled wave are.
  int32_t split_k, n_whole, n_tail;
  float* ws_splitk;
  // Two-SM kernel only: nullptr (pair p takes units p, p + pairs, ...) or a list balanced by cost:
  // [0, pairs] offsets into this same array, then the units of each pair (sched_pairs = the pair count
  // the list was made for).
  const int32_t* unit_list;
  int32_t sched_pairs;
  // Two-SM kernel, plans made with per-adapter ranks (all null otherwise): columns of each 256-row tile's low-rank
  // operand, and its B-side rows as 16-row pieces of the adapters' matrices (piece_src = adapter << 8 | row / 16)
  // in column order; the low-rank tensor map then has 16-row boxes.
  const int32_t* tile_cols;
  const int32_t* tile_piece_off;
  const int32_t* piece_src;
  const int32_t* row_grp;        // [M] group of the row inside its 128-row tile, -1: none
  const int32_t* row_adapter;    // [M]
  const int32_t* tile_grp_off;   // [n_mtiles + 1]
  const int32_t* grp_adapter;    // adapters of the groups
  const float* P;                // [M, R] fp32
  const float* scale;            // [n_adapters] or nullptr (P already scaled)
  int32_t* status;               // device status word
};

__device__ __forceinline__ bool gemm_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  for (uint32_t i = 0; i < GEMM_SPIN_LIMIT; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(status, (int32_t)MLORA_ERR_DEVICE_TIMEOUT);
  return false;
}

// Work unit -> (row tile, first output column, width in columns).
__device__ __forceinline__ void gemm_unit(const GemmArgs& args, int unit, int& mt, int& n0, int& nw) {
  int tile = unit, half = 0;
  nw = GEMM_BN;
  if (unit >= args.n_full) {
    tile = args.n_full + ((unit - args.n_full) >> 1);
    half = (unit - args.n_full) & 1;
    nw = GEMM_BN / 2;
  }
  mt = tile % args.n_mtiles;
  n0 = (tile / args.n_mtiles) * GEMM_BN + half * (GEMM_BN / 2);
}

template <int R, bool W_KMAJOR>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_lora_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmL, const __grid_constant__ CUtensorMap tmOut,
                 const GemmArgs args) {
  static_assert(R == 8 || R == 16 || R == 32 || R == 64 || R == 128, "rank");
  constexpr int GPC = R <= 64 ? 64 / R : 1;          // groups per 64-wide low-rank block

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

  const uint32_t sA0 = smem_base;                                   // stage s: sA0 + s * STAGE_BYTES
  const uint32_t sEpi = smem_base + GEMM_STAGES * GEMM_STAGE_BYTES;
  const uint32_t sBar = sEpi + GEMM_EPI_BYTES;
  // barriers: full[S] | empty[S] | lora_full[S] | lora_go[S] | tmem_full[2] | tmem_empty[2]
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (GEMM_STAGES + s); };
  auto bar_lora = [&](int s) { return sBar + 8u * (2 * GEMM_STAGES + s); };
  auto bar_go = [&](int s) { return sBar + 8u * (3 * GEMM_STAGES + s); };
  auto bar_tfull = [&](int b) { return sBar + 8u * (4 * GEMM_STAGES + b); };
  auto bar_tempty = [&](int b) { return sBar + 8u * (4 * GEMM_STAGES + 2 + b); };
  const uint32_t sMisc = sBar + 8u * (4 * GEMM_STAGES + 4);
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_gen + (sMisc - smem_base));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + (sMisc - smem_base) + 8);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < GEMM_STAGES; ++s) {
      ptx::mbar_init(bar_full(s), 1);
      ptx::mbar_init(bar_empty(s), 1);
      ptx::mbar_init(bar_lora(s), 4);
      ptx::mbar_init(bar_go(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(bar_tfull(b), 1);
      ptx::mbar_init(bar_tempty(b), 4);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmIn);
    ptx::prefetch_tmap(&tmW);
    ptx::prefetch_tmap(&tmL);
    ptx::prefetch_tmap(&tmOut);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), GEMM_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  // set-up (barriers, tensor memory, descriptor prefetch) may overlap the predecessor's tail;
  // its outputs (In, P) are first touched below
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();

  const int KB = (args.K + GEMM_BK - 1) / GEMM_BK;
  const int n_units = args.n_units;

  auto tile_groups = [&](int mt) -> int {
    return args.lora_enabled ? (args.tile_grp_off[mt + 1] - args.tile_grp_off[mt]) : 0;
  };

  if (warp == 0) {
    // ============================ TMA producer ============================
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
        int mt, n0, nw;
        gemm_unit(args, unit, mt, n0, nw);
        const int m0 = mt * GEMM_BM;
        const int nbox = nw / 64;                      // 64-column boxes of the B operand
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % GEMM_STAGES;
          if (!(ok = gemm_wait(bar_empty(s), ((it / GEMM_STAGES) & 1) ^ 1, abort_flag, args.status))) break;
          const uint32_t a = sA0 + s * GEMM_STAGE_BYTES, b = a + GEMM_A_BYTES;
          ptx::mbar_arrive_expect_tx(bar_full(s), GEMM_A_BYTES + (uint32_t)nw * GEMM_BK * 2u);
          ptx::tma_load_2d(a, &tmIn, kb * GEMM_BK, m0, bar_full(s));
          // the B operand arrives in halves of 128 output columns (one TMA each)
          if (W_KMAJOR) {                              // [N, K]: box of 128 rows x 64 k
            ptx::tma_load_2d(b, &tmW, kb * GEMM_BK, n0, bar_full(s));
            if (nw == GEMM_BN) ptx::tma_load_2d(b + 16384, &tmW, kb * GEMM_BK, n0 + 128, bar_full(s));
          } else {                                     // [K, N] seen as (64 n, K, N / 64): box 64 x 64 k x 2
            ptx::tma_load_3d(b, &tmW, 0, kb * GEMM_BK, n0 >> 6, bar_full(s));
            if (nw == GEMM_BN) ptx::tma_load_3d(b + 16384, &tmW, 0, kb * GEMM_BK, (n0 >> 6) + 2, bar_full(s));
          }
        }
        if (!ok) break;
        const int G = tile_groups(mt);
        const int LC = (G * R + 63) / 64;
        const int32_t* ga = args.grp_adapter + (args.lora_enabled ? args.tile_grp_off[mt] : 0);
        for (int lc = 0; lc < LC; ++lc, ++it) {
          const int s = it % GEMM_STAGES;
          if (!(ok = gemm_wait(bar_empty(s), ((it / GEMM_STAGES) & 1) ^ 1, abort_flag, args.status))) break;
          // The operand builders cannot wait on empty[s] themselves: they reach this point a whole
          // main loop early, and a parity wait that lags by more than one phase aliases.  The
          // producer, which follows the ring in order, hands the free slot over instead.
          ptx::mbar_arrive(bar_go(s));
          const uint32_t b = sA0 + s * GEMM_STAGE_BYTES + GEMM_A_BYTES;
          if (R <= 64) {
            const int g0 = lc * GPC;
            int ng = G - g0 < GPC ? G - g0 : GPC;
            // a half-filled 16-deep MMA step (rank 8, odd group count) is padded with a second
            // copy of the last group: its A columns are zero, so it only has to be finite
            const int ngl = (R == 8 && (ng & 1)) ? ng + 1 : ng;
            ptx::mbar_arrive_expect_tx(bar_full(s), (uint32_t)ngl * R * 128u * (uint32_t)nbox);
            for (int i = 0; i < ngl; ++i) {
              const int adapter = ga[g0 + (i < ng ? i : ng - 1)];
              // one box per 64-column block: block nb of the stage starts at nb * 8 KiB
              for (int nb = 0; nb < nbox; ++nb)
                ptx::tma_load_3d(b + nb * 8192 + i * R * 128, &tmL, 0, adapter * R, (n0 >> 6) + nb, bar_full(s));
            }
          } else {
            const int adapter = ga[lc >> 1];
            ptx::mbar_arrive_expect_tx(bar_full(s), 64u * 128u * (uint32_t)nbox);
            for (int nb = 0; nb < nbox; ++nb)
              ptx::tma_load_3d(b + nb * 8192, &tmL, 0, adapter * R + (lc & 1) * 64, (n0 >> 6) + nb, bar_full(s));
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ============================ MMA issuer ============================
    if (lane == 0) {
      constexpr uint32_t idesc_main_full = ptx::make_idesc_bf16(GEMM_BM, GEMM_BN, false, !W_KMAJOR);
      constexpr uint32_t idesc_lora_full = ptx::make_idesc_bf16(GEMM_BM, GEMM_BN, false, true);
      constexpr uint32_t idesc_main_half = ptx::make_idesc_bf16(GEMM_BM, GEMM_BN / 2, false, !W_KMAJOR);
      constexpr uint32_t idesc_lora_half = ptx::make_idesc_bf16(GEMM_BM, GEMM_BN / 2, false, true);
      uint32_t it = 0, lt = 0, lora_phase = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x, ++lt) {
        int mt, n0, nw;
        gemm_unit(args, unit, mt, n0, nw);
        const uint32_t idesc_main = nw == GEMM_BN ? idesc_main_full : idesc_main_half;
        const uint32_t idesc_lora = nw == GEMM_BN ? idesc_lora_full : idesc_lora_half;
        const uint32_t buf = lt & 1;
        if (!(ok = gemm_wait(bar_tempty(buf), ((lt >> 1) & 1) ^ 1, abort_flag, args.status))) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * GEMM_BN;
        uint32_t acc = 0;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % GEMM_STAGES;
          if (!(ok = gemm_wait(bar_full(s), (it / GEMM_STAGES) & 1, abort_flag, args.status))) break;
          ptx::tc_fence_after();
          const uint32_t a = sA0 + s * GEMM_STAGE_BYTES, b = a + GEMM_A_BYTES;
          const uint64_t adesc = ptx::make_smem_desc(a, 16, 1024);
          const uint64_t bdesc = W_KMAJOR ? ptx::make_smem_desc(b, 16, 1024) : ptx::make_smem_desc(b, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < GEMM_BK / 16; ++ks) {
            // K-major: 16 elements = 32 B further along the swizzled row; MN-major: 16 K-rows = 2 KiB
            const uint64_t ad = adesc + (uint64_t)(ks * 2);
            const uint64_t bd = bdesc + (uint64_t)(W_KMAJOR ? ks * 2 : ks * 128);
            ptx::umma_f16(d_tmem, ad, bd, idesc_main, acc);
            acc = 1;
          }
          ptx::umma_commit(bar_empty(s));
        }
        if (!ok) break;
        const int G = tile_groups(mt);
        const int LC = (G * R + 63) / 64;
        for (int lc = 0; lc < LC; ++lc, ++it) {
          const int s = it % GEMM_STAGES;
          if (!(ok = gemm_wait(bar_full(s), (it / GEMM_STAGES) & 1, abort_flag, args.status))) break;
          if (!(ok = gemm_wait(bar_lora(s), (lora_phase >> s) & 1, abort_flag, args.status))) break;
          lora_phase ^= 1u << s;
          ptx::tc_fence_after();
          const uint32_t a = sA0 + s * GEMM_STAGE_BYTES, b = a + GEMM_A_BYTES;
          const uint64_t adesc = ptx::make_smem_desc(a, 16, 1024);
          const uint64_t bdesc = ptx::make_smem_desc(b, 8192, 1024);
          int ksteps = (G * R - lc * 64 + 15) / 16;
          ksteps = ksteps < 4 ? ksteps : 4;
          for (int ks = 0; ks < ksteps; ++ks) {
            ptx::umma_f16(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 128), idesc_lora, acc);
            acc = 1;
          }
          ptx::umma_commit(bar_empty(s));
        }
        if (!ok) break;
        ptx::umma_commit(bar_tfull(buf));
      }
    }
    __syncwarp();
  } else if (warp < 6) {
    // ============================ epilogue ============================
    const int e = warp & 3;                         // tensor-memory lane quarter this warp may read
    const uint32_t stage0 = sEpi + (uint32_t)(warp - 2) * 8192u;
    uint32_t lt = 0;
    bool ok = true;
    for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x, ++lt) {
      int mt, n0, nw;
      gemm_unit(args, unit, mt, n0, nw);
      const int m0 = mt * GEMM_BM + e * 32;
      const int nchunks = nw / 64;
      const uint32_t buf = lt & 1;
      if (!(ok = gemm_wait(bar_tfull(buf), (lt >> 1) & 1, abort_flag, args.status))) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + buf * GEMM_BN + ((uint32_t)(e * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < nchunks; ++c) {
        uint32_t v0[32], v1[32];
        ptx::tmem_ld_32x32b_x32(taddr + c * 64, v0);
        ptx::tmem_ld_32x32b_x32(taddr + c * 64 + 32, v1);
        ptx::tmem_ld_wait();
        if (c == nchunks - 1) {                     // accumulator fully read: hand it back
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar_tempty(buf));
        }
        const uint32_t sb = stage0 + (uint32_t)(c & 1) * 4096u;
        if (lane == 0) ptx::tma_store_wait_read<1>();   // the store that last used this buffer has read it
        __syncwarp();
        const uint32_t rowaddr = sb + (uint32_t)lane * 128u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t p0 = ptx::pack_bf16(__uint_as_float(v0[8 * j + 0]), __uint_as_float(v0[8 * j + 1]));
          const uint32_t p1 = ptx::pack_bf16(__uint_as_float(v0[8 * j + 2]), __uint_as_float(v0[8 * j + 3]));
          const uint32_t p2 = ptx::pack_bf16(__uint_as_float(v0[8 * j + 4]), __uint_as_float(v0[8 * j + 5]));
          const uint32_t p3 = ptx::pack_bf16(__uint_as_float(v0[8 * j + 6]), __uint_as_float(v0[8 * j + 7]));
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rowaddr + (uint32_t)((j ^ (lane & 7)) << 4)),
                       "r"(p0), "r"(p1), "r"(p2), "r"(p3) : "memory");
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t p0 = ptx::pack_bf16(__uint_as_float(v1[8 * j + 0]), __uint_as_float(v1[8 * j + 1]));
          const uint32_t p1 = ptx::pack_bf16(__uint_as_float(v1[8 * j + 2]), __uint_as_float(v1[8 * j + 3]));
          const uint32_t p2 = ptx::pack_bf16(__uint_as_float(v1[8 * j + 4]), __uint_as_float(v1[8 * j + 5]));
          const uint32_t p3 = ptx::pack_bf16(__uint_as_float(v1[8 * j + 6]), __uint_as_float(v1[8 * j + 7]));
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rowaddr + (uint32_t)(((4 + j) ^ (lane & 7)) << 4)),
                       "r"(p0), "r"(p1), "r"(p2), "r"(p3) : "memory");
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        // One group per chunk, empty for a chunk past the edge: the wait above counts groups, so a
        // skipped commit would let the chunk after next reuse a buffer whose store is still reading.
        if (lane == 0) {
          if (m0 < args.M && n0 + c * 64 < args.N)
            ptx::tma_store_2d(&tmOut, sb, n0 + c * 64, m0);   // rows / columns past the edge are clipped
          ptx::tma_store_commit();
        }
      }
    }
    if (lane == 0) ptx::tma_store_wait<0>();
    __syncwarp();
  } else {
    // ============================ low-rank operand builder ============================
    const int rloc = (warp - 6) * 32 + lane;        // row inside the tile
    uint32_t it = 0, go_phase = 0;
    bool ok = true;
    for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
      int mt, n0, nw;
      gemm_unit(args, unit, mt, n0, nw);
      const int G = tile_groups(mt);
      const int LC = (G * R + 63) / 64;
      it += KB;
      if (LC == 0) continue;
      const int row = mt * GEMM_BM + rloc;
      const int grp = row < args.M ? args.row_grp[row] : -1;
      uint32_t ub[R / 2];
      if (grp >= 0) {
        const float sc = args.scale ? args.scale[args.row_adapter[row]] : 1.0f;
        const float4* src = reinterpret_cast<const float4*>(args.P + (size_t)row * R);
#pragma unroll
        for (int i = 0; i < R / 4; ++i) {
          const float4 f = src[i];
          ub[2 * i] = ptx::pack_bf16(f.x * sc, f.y * sc);
          ub[2 * i + 1] = ptx::pack_bf16(f.z * sc, f.w * sc);
        }
      } else {
#pragma unroll
        for (int i = 0; i < R / 2; ++i) ub[i] = 0;
      }
      for (int lc = 0; lc < LC; ++lc, ++it) {
        const int s = it % GEMM_STAGES;
        if (!(ok = gemm_wait(bar_go(s), (go_phase >> s) & 1, abort_flag, args.status))) break;
        go_phase ^= 1u << s;
        const uint32_t rowaddr = sA0 + s * GEMM_STAGE_BYTES + (uint32_t)rloc * 128u;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint32_t w0 = 0, w1 = 0, w2 = 0, w3 = 0;
          if constexpr (R <= 64) {
            const int gg = lc * GPC + (c * 8) / R;
            constexpr int dummy_r = R;   // (c * 8) % R is a compile-time value once c is unrolled
            const int o = ((c * 8) % dummy_r) / 2;
            if (grp == gg) { w0 = ub[o]; w1 = ub[o + 1]; w2 = ub[o + 2]; w3 = ub[o + 3]; }
          } else {
            if (grp == (lc >> 1)) {
              if (lc & 1) { w0 = ub[R / 4 + c * 4]; w1 = ub[R / 4 + c * 4 + 1]; w2 = ub[R / 4 + c * 4 + 2]; w3 = ub[R / 4 + c * 4 + 3]; }
              else        { w0 = ub[c * 4]; w1 = ub[c * 4 + 1]; w2 = ub[c * 4 + 2]; w3 = ub[c * 4 + 3]; }
            }
          }
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rowaddr + (uint32_t)((c ^ (rloc & 7)) << 4)),
                       "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_lora(s));
      }
    }
  }

  // ============================ common exit ============================
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, GEMM_TMEM_COLS);
  }
}

}  // namespace mlora
