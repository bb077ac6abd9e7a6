// Two-SM variant of the fused GEMM + LoRA-expand kernel (see gemm_tcgen05.cuh for the operator).
//
// Two CTAs of a cluster (a pair of SMs) share one 256 x 256 output tile with tcgen05.mma
// cta_group::2: CTA r of the pair owns rows [128 r, 128 r + 128) of the tile (its A operand and
// its accumulator, 128 lanes x 256 columns of its own tensor memory) and supplies columns
// [128 r, 128 r + 128) of the B operand; the tensor cores of both SMs read both halves of B.
// Per output element this moves a third less data from L2 into shared memory than two
// independent 128 x 256 tiles, which is what bounds the one-SM kernel.  No load is multicast:
// every CTA fetches exactly the bytes that land in its own shared memory.
//
// The low-rank part needs no software-built operand here: the shrink kernel has already written
// the rows' scaled rank-R values as block-diagonal bf16 chunks of [256 rows][64] (see PbdArgs), so
// an extra K-block is an ordinary stage - A tile from that buffer, B tile = the groups' expand
// matrices - and the CTA has only three roles (TMA producer, MMA issuer, four epilogue warps).
//
// Synchronisation across the pair (rank 0 = leader, the only issuer of MMAs):
//   full[s]       in the leader: leader's producer arrives with the byte count of BOTH CTAs;
//                 both CTAs' TMA loads complete on it (cta_group::2 loads may signal the peer).
//   empty[s]      in each CTA: tcgen05.commit multicast to both (releases both producers).
//   tmem_full[b]  in each CTA: tcgen05.commit multicast (wakes both epilogues).
//   tmem_empty[b] in the leader: 8 arrivals = 4 epilogue warps x 2 CTAs.
// Every wait is bounded; the pair leaves through a cluster barrier before tensor memory is freed,
// so neither CTA exits while the other may still touch its shared memory.
#pragma once

#include <cuda.h>

#include "gemm_tcgen05.cuh"
#include "ptx.cuh"

namespace mlora {

constexpr int GEMM2_BM = 256;                 // rows of a pair tile (128 per CTA)
constexpr int GEMM2_BN = 256;
constexpr int GEMM2_STAGES = 6;
constexpr int GEMM2_THREADS = 192;          // producer warp, MMA warp, four epilogue warps
constexpr uint32_t GEMM2_A_BYTES = 128 * GEMM_BK * 2;               // 16 KiB: this CTA's rows
constexpr uint32_t GEMM2_B_BYTES = 128 * GEMM_BK * 2;               // 16 KiB: this CTA's half of B
constexpr uint32_t GEMM2_STAGE_BYTES = GEMM2_A_BYTES + GEMM2_B_BYTES;
constexpr uint32_t GEMM2_SMEM_BYTES = GEMM2_STAGES * GEMM2_STAGE_BYTES + GEMM_EPI_BYTES + 512 + 1024 + 1024;

namespace ptx {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on an mbarrier given by a shared::cluster address (possibly in the peer CTA).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 P, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Tiled loads of a CTA pair: data lands in the executing CTA, completion is counted on `bar`,
// a shared::cluster address that may name the peer's barrier.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const void* tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const void* tmap, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem2_alloc(uint32_t smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem2_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem2_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once every
// tcgen05 operation issued so far by this thread is done.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}\n"
      ::"r"(bar) : "memory");
}

}  // namespace ptx

__device__ __forceinline__ bool gemm2_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  for (uint32_t i = 0; i < GEMM_SPIN_LIMIT; ++i) {
    if (ptx::mbar_try_wait_cluster(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(status, (int32_t)MLORA_ERR_DEVICE_TIMEOUT);
  return false;
}

// Tile order: m-fastest inside bands of `group_m` row tiles (all row tiles when group_m == 0), so
// that the tiles in flight at one time cover a near-square block of the output and the operand
// panels they stream together are as few as possible.
__host__ __device__ __forceinline__ void gemm2_tile(const GemmArgs& args, int tile, int& mt, int& nt) {
  const int gm_full = args.group_m > 0 ? args.group_m : args.n_mtiles;
  const int band_tiles = gm_full * args.n_ntiles;
  const int band = tile / band_tiles, r = tile - band * band_tiles;
  const int left = args.n_mtiles - band * gm_full;
  const int gm = left < gm_full ? left : gm_full;
  mt = band * gm_full + r % gm;
  nt = r / gm;
}

// Work unit -> (tile, K slice, slices of that tile).
__host__ __device__ __forceinline__ void gemm2_unit(const GemmArgs& args, int unit, int& tile, int& ks, int& sk) {
  if (unit < args.n_whole) { tile = unit; ks = 0; sk = 1; return; }
  const int u = unit - args.n_whole;
  ks = u / args.n_tail;
  tile = args.n_whole + u - ks * args.n_tail;
  sk = args.split_k;
}

// args: n_mtiles counts 256-row pair tiles, n_ntiles 256-column tiles, n_units = n_whole + n_tail * split_k;
// row_grp / tile_grp_off / grp_adapter are the tables for 256-row tiles.
template <int R, bool W_KMAJOR>
__global__ void __launch_bounds__(GEMM2_THREADS, 1)
gemm2_lora_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmW,
                  const __grid_constant__ CUtensorMap tmL, const __grid_constant__ CUtensorMap tmOut,
                  const __grid_constant__ CUtensorMap tmPbd, const GemmArgs args) {
  static_assert(R == 8 || R == 16 || R == 32 || R == 64 || R == 128, "rank");
  constexpr int GPC = R <= 64 ? 64 / R : 1;          // groups per 64-wide low-rank block
  constexpr int S = GEMM2_STAGES;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

  const uint32_t sA0 = smem_base;
  const uint32_t sEpi = smem_base + S * GEMM2_STAGE_BYTES;
  const uint32_t sBar = sEpi + GEMM_EPI_BYTES;
  // barriers: full[S] | empty[S] | tmem_full[2] | tmem_empty[2]
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (S + s); };
  auto bar_tfull = [&](int b) { return sBar + 8u * (2 * S + b); };
  auto bar_tempty = [&](int b) { return sBar + 8u * (2 * S + 2 + b); };
  const uint32_t sMisc = sBar + 8u * (2 * S + 4);
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_gen + (sMisc - smem_base));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + (sMisc - smem_base) + 8);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();     // 0: leader
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      ptx::mbar_init(bar_full(s), 1);
      ptx::mbar_init(bar_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(bar_tfull(b), 1);
      ptx::mbar_init(bar_tempty(b), 8);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmIn);
    ptx::prefetch_tmap(&tmW);
    ptx::prefetch_tmap(&tmL);
    ptx::prefetch_tmap(&tmOut);
    ptx::prefetch_tmap(&tmPbd);
  }
  if (warp == 1) {                                   // the same warp in both CTAs
    ptx::tmem2_alloc(ptx::smem_u32(tmem_ptr_smem), GEMM_TMEM_COLS);
    ptx::tmem2_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();                           // the peer's barriers exist from here on
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();

  const int KB = (args.K + GEMM_BK - 1) / GEMM_BK;
  const int n_units = args.n_units;
  const int n_pairs = gridDim.x >> 1;
  const int pair = blockIdx.x >> 1;
  // Units of this pair: every n_pairs-th one, or - when the tiles differ in cost (adapter-heavy row tiles) -
  // entries [unit_list[pair], unit_list[pair + 1]) of a list the host balanced by cost.
  const int32_t* ulist = args.unit_list;
  const int u_begin = ulist ? ulist[pair] : pair;
  const int u_end = ulist ? ulist[pair + 1] : n_units;
  const int u_step = ulist ? 1 : n_pairs;

  auto tile_groups = [&](int mt) -> int {
    return args.lora_enabled ? (args.tile_grp_off[mt + 1] - args.tile_grp_off[mt]) : 0;
  };

  if (warp == 0) {
    // ============================ TMA producer (both CTAs) ============================
    // Lane 0 waits and issues the main loads; the low-rank stages are issued by all lanes, one
    // adapter group per lane, from a copy of the tile's adapter list in shared memory, so that
    // the list costs one memory latency per tile rather than one per group.
    int32_t* ga_smem = reinterpret_cast<int32_t*>(smem_gen + (sMisc - smem_base) + 64);   // 256 entries
    uint32_t it = 0;
    bool ok = true;
    for (int ui = u_begin; ui < u_end && ok; ui += u_step) {
      const int unit = ulist ? ulist[ui] : ui;
      int tile, ks, SK;
      gemm2_unit(args, unit, tile, ks, SK);
      int mt, nt;
      gemm2_tile(args, tile, mt, nt);
      const int m0 = mt * GEMM2_BM + (int)rank * 128;
      const int nh = nt * GEMM2_BN + (int)rank * 128;     // this CTA's half of the B columns
      const int G = tile_groups(mt);
      const bool ranked = args.piece_src != nullptr && args.lora_enabled;
      const int LC = ((ranked ? args.tile_cols[mt] : G * R) + 63) / 64;
      const int pc_base = ranked ? args.tile_piece_off[mt] : 0, pc_end = ranked ? args.tile_piece_off[mt + 1] : 0;
      // a K slice takes its share of the low-rank blocks as well (an adapter-heavy tile has more of them than K-blocks)
      const int lc_begin = (int)((long long)ks * LC / SK), lc_end = (int)((long long)(ks + 1) * LC / SK);
      const int kb_begin = (int)((long long)ks * KB / SK), kb_end = (int)((long long)(ks + 1) * KB / SK);
      const int chunk_base = args.lora_enabled ? args.tile_grp_off[mt] : 0;   // chunk slot = 2 * this + lc
      int32_t ga_reg[8];                                  // G <= 256 adapters of the pair tile
      {
        const int32_t* ga = args.grp_adapter + (args.lora_enabled ? args.tile_grp_off[mt] : 0);
#pragma unroll
        for (int j = 0; j < 8; ++j) ga_reg[j] = (lane + 32 * j < G) ? ga[lane + 32 * j] : 0;
      }
      for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
        const int s = it % S;
        if (lane == 0) {
          ok = gemm2_wait(bar_empty(s), ((it / S) & 1) ^ 1, abort_flag, args.status);
          if (ok) {
            const uint32_t a = sA0 + s * GEMM2_STAGE_BYTES, b = a + GEMM2_A_BYTES;
            const uint32_t full = ptx::map_to_cta(bar_full(s), 0);
            if (leader) ptx::mbar_arrive_expect_tx(bar_full(s), 2 * GEMM2_STAGE_BYTES);
            ptx::tma2_load_2d(a, &tmIn, kb * GEMM_BK, m0, full);
            if (W_KMAJOR) ptx::tma2_load_2d(b, &tmW, kb * GEMM_BK, nh, full);          // [N, K]: 128 rows x 64 k
            else          ptx::tma2_load_3d(b, &tmW, 0, kb * GEMM_BK, nh >> 6, full);  // (64 n, K, N/64): 64 x 64 k x 2
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
      }
      if (!ok) break;
      if (lc_end > lc_begin && !ranked) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (lane + 32 * j < G) ga_smem[lane + 32 * j] = ga_reg[j];
        __syncwarp();
      }
      // ranked plans: the pieces of eight chunks at a time, one per lane (one memory latency per eight chunks, the next
      // eight already on their way)
      auto piece_batch = [&](int first_chunk) -> int {
        const int idx = pc_base + 4 * first_chunk + lane;
        return (ranked && idx < pc_end) ? args.piece_src[idx] : 0;
      };
      int pb_chunk0 = lc_begin & ~7;
      int pb_cur = piece_batch(pb_chunk0), pb_next = piece_batch(pb_chunk0 + 8);
      for (int lc = lc_begin; lc < lc_end; ++lc, ++it) {
        const int s = it % S;
        if (lane == 0) ok = gemm2_wait(bar_empty(s), ((it / S) & 1) ^ 1, abort_flag, args.status);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (ranked && (lc & ~7) != pb_chunk0) { pb_chunk0 += 8; pb_cur = pb_next; pb_next = piece_batch(pb_chunk0 + 8); }
        const int piece_of_lane = __shfl_sync(0xffffffffu, pb_cur, 4 * (lc & 7) + (lane & 3));
        const uint32_t a = sA0 + s * GEMM2_STAGE_BYTES, b = a + GEMM2_A_BYTES;
        const uint32_t full = ptx::map_to_cta(bar_full(s), 0);
        // A operand: this CTA's 128 rows of chunk lc of the tile's block-diagonal low-rank matrix
        if (lane == 0) ptx::tma2_load_2d(a, &tmPbd, 0, (2 * chunk_base + lc) * 256 + (int)rank * 128, full);
        if (ranked) {
          // B operand: up to four 16-row pieces of the adapters' matrices, one per lane (tmL has 16-row boxes here)
          const int left = pc_end - (pc_base + 4 * lc);
          const int np = left < 4 ? left : 4;
          if (leader && lane == 0) ptx::mbar_arrive_expect_tx(bar_full(s), 2u * (GEMM2_A_BYTES + (uint32_t)np * 16u * 128u * 2u));
          if (lane < np) {
            const int src = piece_of_lane;
            const int brow = (src >> 8) * R + (src & 255) * 16;
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
              ptx::tma2_load_3d(b + nb * 8192 + lane * 16 * 128, &tmL, 0, brow, (nh >> 6) + nb, full);
          }
        } else if (R <= 64) {
          const int g0 = lc * GPC;
          const int ng = G - g0 < GPC ? G - g0 : GPC;
          const int ngl = (R == 8 && (ng & 1)) ? ng + 1 : ng;   // rank 8: pad a half-filled MMA step
          if (leader && lane == 0) ptx::mbar_arrive_expect_tx(bar_full(s), 2u * (GEMM2_A_BYTES + (uint32_t)ngl * R * 128u * 2u));
          if (lane < ngl) {
            const int adapter = ga_smem[g0 + (lane < ng ? lane : ng - 1)];
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
              ptx::tma2_load_3d(b + nb * 8192 + lane * R * 128, &tmL, 0, adapter * R, (nh >> 6) + nb, full);
          }
        } else {
          if (leader && lane == 0) ptx::mbar_arrive_expect_tx(bar_full(s), 2u * (GEMM2_A_BYTES + 64u * 128u * 2u));
          if (lane < 2)
            ptx::tma2_load_3d(b + lane * 8192, &tmL, 0, ga_smem[lc >> 1] * R + (lc & 1) * 64, (nh >> 6) + lane, full);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ============================ MMA issuer (leader only) ============================
    if (leader && lane == 0) {
      constexpr uint32_t idesc_main = ptx::make_idesc_bf16(GEMM2_BM, GEMM2_BN, false, !W_KMAJOR);
      constexpr uint32_t idesc_lora = ptx::make_idesc_bf16(GEMM2_BM, GEMM2_BN, false, true);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int ui = u_begin; ui < u_end && ok; ui += u_step, ++lt) {
        const int unit = ulist ? ulist[ui] : ui;
        int tile, ks, SK;
        gemm2_unit(args, unit, tile, ks, SK);
        int mt, nt_unused;
        gemm2_tile(args, tile, mt, nt_unused);
        const int kb_begin = (int)((long long)ks * KB / SK), kb_end = (int)((long long)(ks + 1) * KB / SK);
        // columns of the tile's low-rank operand (read here, so that the main loop hides the latency)
        const int lcols = (args.piece_src != nullptr && args.lora_enabled) ? args.tile_cols[mt] : tile_groups(mt) * R;
        const uint32_t buf = lt & 1;
        if (!(ok = gemm2_wait(bar_tempty(buf), ((lt >> 1) & 1) ^ 1, abort_flag, args.status))) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * GEMM2_BN;
        uint32_t acc = 0;
        for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
          const int s = it % S;
          if (!(ok = gemm2_wait(bar_full(s), (it / S) & 1, abort_flag, args.status))) break;
          ptx::tc_fence_after();
          const uint32_t a = sA0 + s * GEMM2_STAGE_BYTES, b = a + GEMM2_A_BYTES;
          const uint64_t adesc = ptx::make_smem_desc(a, 16, 1024);
          const uint64_t bdesc = W_KMAJOR ? ptx::make_smem_desc(b, 16, 1024) : ptx::make_smem_desc(b, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < GEMM_BK / 16; ++ks) {
            ptx::umma2_f16(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(W_KMAJOR ? ks * 2 : ks * 128),
                           idesc_main, acc);
            acc = 1;
          }
          ptx::umma2_commit_both(bar_empty(s));
        }
        if (!ok) break;
        const int LC = (lcols + 63) / 64;
        const int lc_begin = (int)((long long)ks * LC / SK), lc_end = (int)((long long)(ks + 1) * LC / SK);
        for (int lc = lc_begin; lc < lc_end; ++lc, ++it) {
          const int s = it % S;
          if (!(ok = gemm2_wait(bar_full(s), (it / S) & 1, abort_flag, args.status))) break;
          ptx::tc_fence_after();
          const uint32_t a = sA0 + s * GEMM2_STAGE_BYTES, b = a + GEMM2_A_BYTES;
          const uint64_t adesc = ptx::make_smem_desc(a, 16, 1024);
          const uint64_t bdesc = ptx::make_smem_desc(b, 8192, 1024);
          int ksteps = (lcols - lc * 64 + 15) / 16;
          ksteps = ksteps < 4 ? ksteps : 4;
          for (int ks = 0; ks < ksteps; ++ks) {
            ptx::umma2_f16(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 128), idesc_lora, acc);
            acc = 1;
          }
          ptx::umma2_commit_both(bar_empty(s));
        }
        if (!ok) break;
        ptx::umma2_commit_both(bar_tfull(buf));
      }
    }
    __syncwarp();
  } else {
    // ============================ epilogue (both CTAs, own rows) ============================
    const int e = warp & 3;
    const uint32_t stage0 = sEpi + (uint32_t)(warp - 2) * 8192u;
    uint32_t lt = 0;
    bool ok = true;
    for (int ui = u_begin; ui < u_end && ok; ui += u_step, ++lt) {
      const int unit = ulist ? ulist[ui] : ui;
      int tile, ks, SK;
      gemm2_unit(args, unit, tile, ks, SK);
      int mt, nt;
      gemm2_tile(args, tile, mt, nt);
      const int m0 = mt * GEMM2_BM + (int)rank * 128 + e * 32, n0 = nt * GEMM2_BN;
      const uint32_t buf = lt & 1;
      if (!(ok = gemm2_wait(bar_tfull(buf), (lt >> 1) & 1, abort_flag, args.status))) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + buf * GEMM2_BN + ((uint32_t)(e * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < GEMM2_BN / 64; ++c) {
        uint32_t v0[32], v1[32];
        ptx::tmem_ld_32x32b_x32(taddr + c * 64, v0);
        ptx::tmem_ld_32x32b_x32(taddr + c * 64 + 32, v1);
        ptx::tmem_ld_wait();
        if (c == GEMM2_BN / 64 - 1) {               // accumulator fully read: tell the leader
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(bar_tempty(buf), 0));
        }
        if (SK > 1) {       // a K slice: this lane's row of the fp32 partial, 64 columns, for the reduction kernel
          const int row = m0 + lane;
          if (row < args.M) {
            float* dst = args.ws_splitk + (((size_t)ks * args.n_tail + (tile - args.n_whole)) * GEMM2_BM +
                                           ((int)rank * 128 + e * 32 + lane)) * GEMM2_BN + c * 64;
            // 256-bit stores: every store fills whole 32-byte sectors of this lane's row
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (n0 + c * 64 + 8 * j < args.N)
                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 8 * j),
                             "r"(v0[8 * j]), "r"(v0[8 * j + 1]), "r"(v0[8 * j + 2]), "r"(v0[8 * j + 3]),
                             "r"(v0[8 * j + 4]), "r"(v0[8 * j + 5]), "r"(v0[8 * j + 6]), "r"(v0[8 * j + 7]) : "memory");
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (n0 + c * 64 + 32 + 8 * j < args.N)
                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 32 + 8 * j),
                             "r"(v1[8 * j]), "r"(v1[8 * j + 1]), "r"(v1[8 * j + 2]), "r"(v1[8 * j + 3]),
                             "r"(v1[8 * j + 4]), "r"(v1[8 * j + 5]), "r"(v1[8 * j + 6]), "r"(v1[8 * j + 7]) : "memory");
          }
          continue;
        }
        const uint32_t sb = stage0 + (uint32_t)(c & 1) * 4096u;
        if (lane == 0) ptx::tma_store_wait_read<1>();
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
          if (m0 < args.M && n0 + c * 64 < args.N) ptx::tma_store_2d(&tmOut, sb, n0 + c * 64, m0);
          ptx::tma_store_commit();
        }
      }
    }
    if (lane == 0) ptx::tma_store_wait<0>();
    __syncwarp();
  }

  // ============================ common exit ============================
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();          // the peer is done with this CTA's shared memory and barriers
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem2_dealloc(tmem_base, GEMM_TMEM_COLS);
  }
}

// Sum of the K slices of the split tiles: Out[m, n] = bf16(sum over slices of the tile's fp32
// partials), slices added in index order.  One thread per 8 columns of a row of a split tile
// (256 x 32 threads per tile); rows and columns past the output's edge are skipped.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const GemmArgs args, __nv_bfloat16* Out, int64_t ld_out) {
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  const int t = blockIdx.x / 32;                                       // split tile
  const int idx = (blockIdx.x % 32) * 256 + threadIdx.x;               // 0 .. 8191
  const int r = idx >> 5, c8 = (idx & 31) * 8;
  int mt, nt;
  gemm2_tile(args, args.n_whole + t, mt, nt);
  const int m = mt * GEMM2_BM + r, n = nt * GEMM2_BN + c8;
  if (m >= args.M || n >= args.N) return;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int s = 0; s < args.split_k; ++s) {
    const float4* src = reinterpret_cast<const float4*>(
        args.ws_splitk + (((size_t)s * args.n_tail + t) * GEMM2_BM + r) * GEMM2_BN + c8);
    const float4 a = src[0], b = src[1];
    acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
    acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
  }
  *reinterpret_cast<uint4*>(Out + (size_t)m * ld_out + n) =
      make_uint4(ptx::pack_bf16(acc[0], acc[1]), ptx::pack_bf16(acc[2], acc[3]), ptx::pack_bf16(acc[4], acc[5]),
                 ptx::pack_bf16(acc[6], acc[7]));
}

}  // namespace mlora
