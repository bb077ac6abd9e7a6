// Rank-r ("skinny") kernels of the multi-LoRA layer for bf16 storage, mma.sync family.  They are bound by
// the bytes of the wide operand they stream once from HBM; the rank-r contraction itself runs on the
// warp-level tensor-core instruction (mma.sync m16n8k16, fp32 accumulate) because at rank 16 and above the
// CUDA cores could not keep up with the memory system.  These are the defaults up to rank 16 and, at every
// rank, wherever the rows pass through registers for a reason: gathered decode rows, the dropout mask.
// Ranks 32 to 128 otherwise run on the tcgen05 kernels of shrink_tc.cuh and grad_tc.cuh.
//
//  shrink : Out[t, q] = sum_k In[t, k] * P_a(t)[q, k]      (U = X A^T  and  V = s dY B^T)
//           work item = up to 32 rows that share one adapter, GATHERED by adapter id (they need not be
//           adjacent: decode rows of one adapter form one item, prefill and fine-tune segments are
//           runs of items); optionally copies the rows of In and the result into the fine-tuning
//           activation buffers on the way.
//           shrink_stream_kernel (rank <= 64): persistent, stages filled by the copy engine;
//           shrink_kernel (every rank; the only mma.sync shrink at rank 128): one CTA per item, operands
//           straight from global memory.
//  grad   : G_g[q, j] = sum_{rows t of slot g} P[t, q] * Q[t, j]   (dB = (s U)^T dY, dA = V^T X)
//           grad_stream_kernel (rank <= 64: both gradients in one launch); grad_kernel (every rank, per strip).
//  expand_mask_kernel : the low-rank part of the input gradient under dropout.
#pragma once

#include "dropout.cuh"
#include "plan.h"
#include "ptx.cuh"

namespace mlora {

constexpr int GRAD_THREADS = 256;

// Block-diagonal low-rank operand of the two-SM GEMM, written by the shrink kernels.  For each
// 256-row tile with G adapter groups the rows' (scaled) rank-R values are laid out as a
// [256, G R] matrix that is zero outside each row's own group block, cut into 64-column chunks of
// [256 rows][64] bf16 (one chunk = the A operand of one extra K-block of the GEMM).  Chunk c of
// tile t lives at chunk slot 2 * tile2_grp_off[t] + c (two slots per group cover rank <= 128).
struct PbdArgs {
  __nv_bfloat16* pbd;            // nullable: [slots * 256, 64]
  const int32_t* row_grp2;       // [rows] group of the row inside its 256-row tile, -1: none
  const int32_t* tile2_grp_off;  // [tiles + 1]
  const float* scale;            // nullable: values multiplied by scale[adapter]
  const int32_t* zero_rows;      // rows without an adapter inside tiles that have groups
  int32_t n_zero_rows;
  // plans made with per-adapter ranks (all three null otherwise: group g of a tile starts at column g R and is R wide)
  const int32_t* grp2_col = nullptr;     // [groups] first column of the group in its tile's operand
  const int32_t* grp2_width = nullptr;   // [groups] its width (the adapter's rank rounded up to 16)
  const int32_t* tile2_cols = nullptr;   // [tiles] columns of the tile's operand
};

// One warp writes all chunks of one row: `vals` = the row's R fp32 values (nullptr: all zero).
// The table entries of the row (first group slot of its tile, groups of the tile, the row's own
// group or -1) are passed in, so that a caller can fetch them long before the values exist.
template <int R>
__device__ __forceinline__ void pbd_write_row_at(const PbdArgs& pa, int row, int goff, int G, int g, const float* vals,
                                                 float sc, int lane) {
  const int rl = row & 255;
  const int cols = pa.tile2_cols ? pa.tile2_cols[row >> 8] : G * R;
  const int LC = (cols + 63) / 64;
  const int c0 = g < 0 ? 0 : (pa.grp2_col ? pa.grp2_col[goff + g] : g * R);        // the row's own columns: [c0, c0 + w)
  const int w = g < 0 ? 0 : (pa.grp2_width ? pa.grp2_width[goff + g] : R);
  for (int piece = lane; piece < LC * 8; piece += 32) {
    const int c = piece >> 3, kcol = piece * 8;          // chunk, first low-rank column of the piece
    uint4 v = make_uint4(0, 0, 0, 0);
    if (kcol >= c0 && kcol < c0 + w) {
      const float4 f0 = *reinterpret_cast<const float4*>(vals + (kcol - c0));
      const float4 f1 = *reinterpret_cast<const float4*>(vals + (kcol - c0) + 4);
      v.x = ptx::pack_bf16(f0.x * sc, f0.y * sc); v.y = ptx::pack_bf16(f0.z * sc, f0.w * sc);
      v.z = ptx::pack_bf16(f1.x * sc, f1.y * sc); v.w = ptx::pack_bf16(f1.z * sc, f1.w * sc);
    }
    __nv_bfloat16* dst = pa.pbd + ((size_t)(2 * goff + c) * 256 + rl) * 64 + (piece & 7) * 8;
    *reinterpret_cast<uint4*>(dst) = v;
  }
}

template <int R>
__device__ __forceinline__ void pbd_write_row(const PbdArgs& pa, int row, const float* vals, float sc, int lane) {
  const int tile = row >> 8;
  const int goff = pa.tile2_grp_off[tile];
  pbd_write_row_at<R>(pa, row, goff, pa.tile2_grp_off[tile + 1] - goff, vals ? pa.row_grp2[row] : -1, vals, sc, lane);
}

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
  const int32_t* item_save;    // nullable: parallel to item_rows, save offset of the row or -1
  __nv_bfloat16* x_save;       // nullable, [cap, D] dense
  float* u_save;               // nullable, [cap, R] dense
  int64_t save_base;
  int64_t save_cap;            // rows of x_save (extent of its tensor map)
  // split of the contraction over gridDim.y CTAs per item (used when there are few items):
  float* partial;              // [n_items * gridDim.z * gridDim.y, MT * 16, R] scratch
  int32_t* counters;           // [n_items * gridDim.z], zero between launches
  PbdArgs pbd;                 // optional block-diagonal copy of the result for the two-SM GEMM
  DropArgs drop = {0, 0, 1.0f}; // per-item kernel with DROP: dropout of the fine-tuning rows' branch input
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
template <int RB, int MT, int WARPS, int MIN_CTAS, bool DROP = false>
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
  const int32_t* saves = a.item_save ? a.item_save + a.item_start[blockIdx.x] + roff : nullptr;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  // this thread's rows: local index g + 8 j, j < 2 MT
  const __nv_bfloat16* xp[2 * MT];
  __nv_bfloat16* sp[2 * MT];
  int msave[2 * MT];             // DROP: save-order place of the row (the mask's row counter), -1: not a fine-tuning row
#pragma unroll
  for (int j = 0; j < 2 * MT; ++j) {
    const int rl = g + 8 * j;
    xp[j] = nullptr; sp[j] = nullptr; msave[j] = -1;
    if (rl < nrows) {
      const int row = rows[rl];
      xp[j] = a.In + (size_t)row * a.ld_in + 16 * c;
      const int sv = (saves && a.x_save) ? saves[rl] : -1;
      if (sv >= 0) sp[j] = a.x_save + (size_t)(a.save_base + sv) * a.D + 16 * c;
      if (DROP && saves) msave[j] = saves[rl];
    }
  }
  const __nv_bfloat16* p0 = a.P_all + ((size_t)adapter * R + g) * a.D + 16 * c;
  // everything above read only the plan's tables; from here on the predecessor's data is touched
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  if (a.pbd.pbd && blockIdx.y == 0 && blockIdx.z == 0)         // rows nobody else owns: all-zero chunks
    for (int i = blockIdx.x * WARPS + warp; i < a.pbd.n_zero_rows; i += gridDim.x * WARPS)
      pbd_write_row<R>(a.pbd, a.pbd.zero_rows[i], nullptr, 0.f, lane);

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
    if (DROP) {      // the saved copy keeps the row as it is, the product does not
#pragma unroll
      for (int j = 0; j < 2 * MT; ++j) {
        if (sp[j]) {
          *reinterpret_cast<uint4*>(sp[j] + ko) = x[j][0];
          *reinterpret_cast<uint4*>(sp[j] + ko + 8) = x[j][1];
        }
        if (msave[j] >= 0) {
          drop_mask8(a.drop, (uint32_t)msave[j], (uint32_t)(ko + 16 * c), x[j][0]);
          drop_mask8(a.drop, (uint32_t)msave[j], (uint32_t)(ko + 16 * c + 8), x[j][1]);
        }
      }
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
      if (!DROP && sp[j]) {
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
    const int sv = saves ? saves[r] : -1;
    if (DROP && sv >= 0) u *= a.drop.keep_scale;
    a.Out[(size_t)row * R + q] = u * sc;
    if (a.u_save && sv >= 0) a.u_save[(size_t)(a.save_base + sv) * R + q] = u;
  }
  if (ksplit > 1 && threadIdx.x == 0) a.counters[item] = 0;     // ready for the next launch
  if (a.pbd.pbd) {
    __syncthreads();             // the rows of Out written above are read back below
    for (int r = warp; r < nrows; r += WARPS) {
      const int row = rows[r];
      pbd_write_row<R>(a.pbd, row, a.Out + (size_t)row * R, a.pbd.scale ? a.pbd.scale[adapter] : 1.0f, lane);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Streaming shrink for ranks up to 32: a persistent grid (one CTA per SM) walks the flattened list
// of work units (item, chunk of 8 K-blocks = 512 elements) in equal contiguous ranges, so every SM
// streams the same number of bytes in one wave.  A producer warp moves each unit into a
// STAGES-deep shared-memory ring, completion counted on an mbarrier: tensor-map tiles of
// 256 elements x 32 rows (16 KiB per instruction) for the adapter rows and for items whose rows
// are adjacent in memory (prefill and fine-tune segments), one bulk copy per row only for items
// gathered from scattered rows (decode rows) - the copy engine's cost is per instruction, not per
// byte.  Eight consumer warps share the K-blocks of the unit: fragments come out of shared memory
// with 16-byte loads, feed mma.sync, and the rows of In are stored on to x_save for fine-tuning
// rows.  Accumulators
// persist across the chunks of an item and are flushed when the item ends.  An item whose chunks
// were shared by several CTAs is finished by whichever of them arrives last, adding the partials
// in CTA order (a fixed order).  Every mbarrier wait is bounded.
constexpr int STREAM_WARPS = 8;      // consumer warps; warp 8 is the producer
constexpr int STREAM_THREADS = (STREAM_WARPS + 1) * 32;
// A unit covers CHUNK K-blocks of 64 (a template parameter: 8 or 16).  Tile layout of a stage:
// CHUNK / 4 boxes of [rows][256 elements]; row-copy layout (gathered items): rows CHUNK * 128 + 16
// bytes apart, so that fragment loads hit distinct banks.
constexpr uint32_t STREAM_SPIN_LIMIT = 1u << 22;


struct StreamArgs {
  ShrinkArgs s;
  int32_t n_items;
  int32_t chunks_per_item;   // ceil(D / (64 CHUNK))
  int32_t n_units;           // n_items * chunks_per_item
  int32_t units_per_cta;     // ceil(n_units / gridDim.x)
  int32_t* status;           // device status word
  const int32_t* item_desc;    // [n_items][kItemDescInts] packed item records (see RowSpace::item_desc)
  int32_t tma_save;            // 1: tmSave covers x_save; full contiguous fine-tuning items are saved as blocks
  DropArgs drop;               // dropout of the fine-tuning rows' branch input (thr == 0: off)
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ bool stream_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                            uint32_t limit = STREAM_SPIN_LIMIT) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(status, (int32_t)MLORA_ERR_DEVICE_TIMEOUT);
  return false;
}

// Self-test of the give-up path shared by every bounded wait: one thread waits, with the helper the
// streaming kernels use, on a barrier that nothing will ever arrive at, for `polls` polls.  The wait
// then runs out, raises the CTA's abort flag, leaves MLORA_ERR_DEVICE_TIMEOUT in the status word and
// the kernel returns normally - no copy is in flight and no tensor memory is held, so nothing has to
// be drained.  A second thread then waits on the same barrier: it finds the abort flag at its first
// look at it and leaves at once, as the other warps of a streaming CTA do.
__global__ void __launch_bounds__(64)
wait_selftest_kernel(int32_t* status, uint32_t polls) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_word = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) stream_wait(ptx::smem_u32(&bar), 0, &abort_word, status, polls);
  __syncthreads();
  if (threadIdx.x == 32) stream_wait(ptx::smem_u32(&bar), 0, &abort_word, status, 512u);
}

template <int RB, int STAGES, int CHUNK, bool DROP>
__global__ void __launch_bounds__(STREAM_THREADS, 1)
shrink_stream_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmP,
                     const __grid_constant__ CUtensorMap tmSave, const StreamArgs sa) {
  constexpr int R = RB * 8;
  constexpr int NBOX = CHUNK / 4;                          // 256-element boxes per unit
  constexpr uint32_t STREAM_PITCH = CHUNK * 128 + 16;     // row-copy layout
  // tile layout of a box: [4 K-blocks][32 rows][128 B], 16-byte pieces swizzled by (row & 7)
  // (the 128-byte swizzle of the tensor maps), so the 8 rows a warp reads at one K offset fall
  // into 8 different bank groups
  constexpr uint32_t XBOX_BYTES = 4 * 32 * 128;
  constexpr uint32_t X_BYTES = ((32 * STREAM_PITCH > NBOX * XBOX_BYTES ? 32 * STREAM_PITCH : NBOX * XBOX_BYTES) + 1023) / 1024 * 1024;
  constexpr uint32_t PBOX_BYTES = 4 * R * 128;            // adapter rows: [4 K-blocks][R rows][128 B], swizzled
  constexpr uint32_t STAGE_BYTES = X_BYTES + NBOX * PBOX_BYTES;
  static_assert(CHUNK % STREAM_WARPS == 0, "each consumer warp takes CHUNK / 8 K-blocks of a unit");
  constexpr int RW = RB >= 8 ? 2 : (RB >= 4 ? 4 : 8);     // reduction buffers (rank 32: two rounds of 4 warps, rank 64: four of 2)
  extern __shared__ __align__(128) uint8_t stream_smem[];
  __shared__ __align__(16) float fin[32][R];             // an item's final rows, read back for the operand chunks
  __shared__ __align__(8) uint64_t bars[2 * STAGES];     // full[STAGES] | empty[STAGES]
  __shared__ int stage_save[STAGES][2];                  // producer only: {first x_save row or -1, k0} of the staged unit
  __shared__ int is_last;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  const ShrinkArgs& a = sa.s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const int u_begin = cta * sa.units_per_cta;
  const int u_end = min(u_begin + sa.units_per_cta, sa.n_units);
  const int KC = sa.chunks_per_item;
  const int nkb = a.D / 64;
  const uint32_t ring = (ptx::smem_u32(stream_smem) + 1023u) & ~1023u;   // swizzled tiles need 1 KiB alignment
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto bar_full = [&](int st) { return bar0 + 8u * st; };
  auto bar_empty = [&](int st) { return bar0 + 8u * (STAGES + st); };
  float (*red)[32][R + 1] = reinterpret_cast<float (*)[32][R + 1]>(
      stream_smem + (ring - ptx::smem_u32(stream_smem)) + STAGES * STAGE_BYTES);

  if (threadIdx.x == 0) {
    for (int st = 0; st < STAGES; ++st) {
      ptx::mbar_init(bar_full(st), 1);
      ptx::mbar_init(bar_empty(st), STREAM_WARPS);
    }
    abort_word = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();

  if (warp == STREAM_WARPS) {
    // ======================= producer =======================
    int item = u_begin / KC, kc = u_begin % KC;
    int cur = -1, nrows = 0, contig = 0, row0 = 0, prow0 = 0, save_row = -1;
    const __nv_bfloat16* src0 = nullptr;     // gathered items: lane l copies the item's row l
    auto set_item = [&](int it) {
      cur = it;
      const int4 d0 = *reinterpret_cast<const int4*>(sa.item_desc + (size_t)it * kItemDescInts);
      const int2 d1 = *reinterpret_cast<const int2*>(sa.item_desc + (size_t)it * kItemDescInts + 4);
      nrows = d0.y;
      contig = d0.w & 1;
      row0 = d1.x;
      save_row = (sa.tma_save && (d0.w & 2)) ? (int)a.save_base + d1.y : -1;
      src0 = (!contig && lane < nrows) ? a.In + (size_t)a.item_rows[d0.x + lane] * a.ld_in : nullptr;
      prow0 = d0.z * R;
    };
    // block save of a staged unit: the tiles of a full fine-tuning item go from shared memory to
    // x_save as they are (one bulk tensor store per 256-element box, lanes 0 .. NBOX-1)
    auto store_unit = [&](int j) -> bool {
      const int sj = j % STAGES;
      const int srow = stage_save[sj][0];
      if (srow < 0) return true;                         // same value in every lane
      bool got = true;
      if (lane == 0) got = stream_wait(bar_full(sj), (j / STAGES) & 1, abort_flag, sa.status);
      got = __shfl_sync(0xffffffffu, got ? 1 : 0, 0) != 0;
      if (!got) return false;
      const int k0 = stage_save[sj][1];
      if (lane < NBOX && k0 + lane * 256 < a.D)
        ptx::tma_store_3d(&tmSave, ring + (uint32_t)sj * STAGE_BYTES + (uint32_t)lane * XBOX_BYTES, 0, srow, (k0 >> 6) + lane * 4);
      ptx::tma_store_commit();
      return true;
    };
    if (u_begin < u_end) set_item(item);
    ptx::prefetch_tmap(&tmIn);
    ptx::prefetch_tmap(&tmP);
    if (sa.tma_save) ptx::prefetch_tmap(&tmSave);
    ptx::grid_dependency_wait();             // only plan tables were read so far
    ptx::grid_launch_dependents();
    bool ok = true;
    int stored = u_begin;                    // units [u_begin, stored) have had their block save issued
    for (int u = u_begin; u < u_end && ok; ++u) {
      const int i = u - u_begin, st = i % STAGES;
      if (item != cur) set_item(item);
      if (lane == 0) ok = stream_wait(bar_empty(st), ((i / STAGES) & 1) ^ 1, abort_flag, sa.status);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      ptx::tma_store_wait_read<0>();         // the stage's previous block save has left shared memory
      __syncwarp();
      const int k0 = kc * (CHUNK * 64);
      const uint32_t row_bytes = (uint32_t)min(CHUNK * 64, a.D - k0) * 2u;
      const uint32_t xbytes = contig ? NBOX * XBOX_BYTES : (uint32_t)nrows * row_bytes;
      if (lane == 0) {
        stage_save[st][0] = save_row;
        stage_save[st][1] = k0;
        ptx::mbar_arrive_expect_tx(bar_full(st), xbytes + NBOX * PBOX_BYTES);
      }
      __syncwarp();
      const uint32_t dst = ring + (uint32_t)st * STAGE_BYTES;
      // lanes 0 .. NBOX-1: one adapter tile each; lanes NBOX .. 2 NBOX-1: one tile of the item's rows
      // (tiles reaching past the tensor's edge are zero-filled and still count their full size)
      if (lane < NBOX) ptx::tma_load_3d(dst + X_BYTES + (uint32_t)lane * PBOX_BYTES, &tmP, 0, prow0, (k0 >> 6) + lane * 4, bar_full(st));
      if (contig) {
        if (lane >= NBOX && lane < 2 * NBOX)
          ptx::tma_load_3d(dst + (uint32_t)(lane - NBOX) * XBOX_BYTES, &tmIn, 0, row0, (k0 >> 6) + (lane - NBOX) * 4, bar_full(st));
      } else if (src0) {
        bulk_load(dst + (uint32_t)lane * STREAM_PITCH, src0 + k0, row_bytes, bar_full(st));
      }
      if (++kc == KC) { kc = 0; ++item; }
      // with the next load in flight, save the oldest staged unit whose data must have been asked for
      if (i >= STAGES - 1) { ok = store_unit(i - (STAGES - 1)); stored = u - (STAGES - 1) + 1; }
    }
    for (int u = stored; u < u_end && ok; ++u) ok = store_unit(u - u_begin);
    ptx::tma_store_wait<0>();                // block saves complete before the CTA ends
  } else {
    // ======================= consumers =======================
    const int g = lane >> 2, c = lane & 3;
    float acc[2][RB][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int i = 0; i < RB; ++i) acc[m][i][0] = acc[m][i][1] = acc[m][i][2] = acc[m][i][3] = 0.f;

    int item = u_begin / KC, kc = u_begin % KC;
    int cur_item = -1, cur_nrows = 0, cur_adapter = 0, cur_contig = 0;
    const int32_t* cur_rows = nullptr;
    const int32_t* cur_saves = nullptr;
    __nv_bfloat16* sp[4] = {nullptr, nullptr, nullptr, nullptr};
    int msave[4] = {-1, -1, -1, -1};       // save-order place of rows g + 8 j (dropout counter), -1: not a fine-tuning row
    // flush-time values fetched when the item starts: element idx = tid + 256 k of the item's
    // [rows][R] result belongs to row idx / R
    int my_row[RB], my_save[RB];
    float my_scale = 1.0f, pb_scale = 1.0f;
    int pb_row[32 / STREAM_WARPS], pb_goff[32 / STREAM_WARPS], pb_G[32 / STREAM_WARPS], pb_g[32 / STREAM_WARPS];
    // this thread's pieces of a K-block: elements 16c .. 16c+15 of the block
    ptx::grid_dependency_wait();
    bool ok = true;
    if (a.pbd.pbd)                                            // rows nobody else owns: all-zero chunks
      for (int i = cta * STREAM_WARPS + warp; i < a.pbd.n_zero_rows; i += gridDim.x * STREAM_WARPS)
        pbd_write_row<R>(a.pbd, a.pbd.zero_rows[i], nullptr, 0.f, lane);

    for (int u = u_begin; u < u_end; ++u) {
      const int i = u - u_begin, st = i % STAGES;
      if (item != cur_item) {
        cur_item = item;
        const int4 d0 = *reinterpret_cast<const int4*>(sa.item_desc + (size_t)item * kItemDescInts);
        cur_nrows = d0.y;
        cur_adapter = d0.z;
        cur_contig = d0.w & 1;
        const bool block_saved = sa.tma_save && (d0.w & 2);   // the producer stores this item's rows
        cur_rows = a.item_rows + d0.x;
        cur_saves = a.item_save ? a.item_save + d0.x : nullptr;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int rl = g + 8 * j;
          msave[j] = (cur_saves && rl < cur_nrows) ? cur_saves[rl] : -1;
          sp[j] = (!block_saved && a.x_save && msave[j] >= 0)
                      ? a.x_save + (size_t)(a.save_base + msave[j]) * a.D + 16 * c : nullptr;
        }
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = ((int)threadIdx.x + k * STREAM_WARPS * 32) / R;
          my_row[k] = r < cur_nrows ? cur_rows[r] : -1;
          my_save[k] = (r < cur_nrows && cur_saves) ? cur_saves[r] : -1;
        }
        my_scale = a.scale ? a.scale[cur_adapter] : 1.0f;
        if (a.pbd.pbd) {     // table entries of the rows whose operand chunks this warp writes at the flush
          pb_scale = a.pbd.scale ? a.pbd.scale[cur_adapter] : 1.0f;
#pragma unroll
          for (int j = 0; j < 32 / STREAM_WARPS; ++j) {
            const int r = warp + STREAM_WARPS * j;
            pb_row[j] = r < cur_nrows ? cur_rows[r] : -1;
            if (pb_row[j] >= 0) {
              const int tile = pb_row[j] >> 8;
              pb_goff[j] = a.pbd.tile2_grp_off[tile];
              pb_G[j] = a.pbd.tile2_grp_off[tile + 1] - pb_goff[j];
              pb_g[j] = a.pbd.row_grp2[pb_row[j]];
            }
          }
        }
      }
      ok = stream_wait(bar_full(st), (i / STAGES) & 1, abort_flag, sa.status);
      if (!ok) break;
#pragma unroll
      for (int kk = 0; kk < CHUNK / STREAM_WARPS; ++kk) {
        const int kb = kc * CHUNK + kk * STREAM_WARPS + warp;
        if (kb >= nkb) continue;
        const int kbl = kk * STREAM_WARPS + warp;            // K-block inside the unit
        const uint32_t stage = ring + (uint32_t)st * STAGE_BYTES;
        // this thread's two 16-byte pieces (2c, 2c+1) of a row's 128-byte K-block; in the tile
        // layout piece i of row r sits at piece i ^ (r & 7), and r & 7 == g for every row read here
        const uint32_t sw0 = (uint32_t)((2 * c) ^ g) << 4, sw1 = (uint32_t)((2 * c + 1) ^ g) << 4;
        uint4 x[4][2];
        if (cur_contig) {        // tile layout [box][K-block][row][128 B]
          const uint32_t xsrc = stage + (uint32_t)(kbl >> 2) * XBOX_BYTES + (uint32_t)(kbl & 3) * 4096u;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t ra = xsrc + (uint32_t)(g + 8 * j) * 128u;
            x[j][0] = lds_v4(ra + sw0);
            x[j][1] = lds_v4(ra + sw1);
          }
        } else {                 // row-copy layout [row][pitch]
          const uint32_t xsrc = stage + (uint32_t)kbl * 128u + (uint32_t)c * 32u;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t ra = xsrc + (uint32_t)(g + 8 * j) * STREAM_PITCH;
            x[j][0] = lds_v4(ra);
            x[j][1] = lds_v4(ra + 16);
          }
        }
        const uint32_t psrc = stage + X_BYTES + (uint32_t)(kbl >> 2) * PBOX_BYTES + (uint32_t)(kbl & 3) * (R * 128u);
        uint4 p[RB][2];
#pragma unroll
        for (int n = 0; n < RB; ++n) {
          const uint32_t rp = psrc + (uint32_t)(8 * n + g) * 128u;
          p[n][0] = lds_v4(rp + sw0);
          p[n][1] = lds_v4(rp + sw1);
        }
        const int ko = kb * 64;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (sp[j]) {     // activation save of rows that are not block-saved: they pass through here exactly once
            // this thread's 32 contiguous bytes of the row as one 256-bit store (a whole sector)
            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(sp[j] + ko),
                         "r"(x[j][0].x), "r"(x[j][0].y), "r"(x[j][0].z), "r"(x[j][0].w),
                         "r"(x[j][1].x), "r"(x[j][1].y), "r"(x[j][1].z), "r"(x[j][1].w) : "memory");
          }
        // rows past the item's end were not copied: keep their stale bytes out of the MMA
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (g + 8 * j >= cur_nrows) { x[j][0] = make_uint4(0, 0, 0, 0); x[j][1] = make_uint4(0, 0, 0, 0); }
        if (DROP) {     // dropout: the saved copy above keeps the row as it is, the product does not
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (msave[j] >= 0) {
              drop_mask8(sa.drop, (uint32_t)msave[j], (uint32_t)(ko + 16 * c), x[j][0]);
              drop_mask8(sa.drop, (uint32_t)msave[j], (uint32_t)(ko + 16 * c + 8), x[j][1]);
            }
        }
#pragma unroll
        for (int n = 0; n < RB; ++n) {
          const uint32_t rp[8] = {p[n][0].x, p[n][0].y, p[n][0].z, p[n][0].w, p[n][1].x, p[n][1].y, p[n][1].z, p[n][1].w};
#pragma unroll
          for (int m = 0; m < 2; ++m) {
            const uint4 &l0 = x[2 * m][0], &l1 = x[2 * m][1], &h0 = x[2 * m + 1][0], &h1 = x[2 * m + 1][1];
            const uint32_t ra[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
            const uint32_t rb[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
#pragma unroll
            for (int s = 0; s < 4; ++s) {
              ptx::mma_bf16_16816(acc[m][n], ra[2 * s], rb[2 * s], ra[2 * s + 1], rb[2 * s + 1], rp[2 * s], rp[2 * s + 1]);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_empty(st));        // the stage's bytes are in registers now

      // ---- flush when the item (or this CTA's range) ends ----
      const bool item_ends = (kc == KC - 1) || (u == u_end - 1);
      const int this_item = item;
      if (++kc == KC) { kc = 0; ++item; }
      if (!item_ends) continue;
#pragma unroll
      for (int round = 0; round < STREAM_WARPS / RW; ++round) {
        if (warp / RW == round) {
          float (*mine)[R + 1] = red[warp % RW];
#pragma unroll
          for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int n = 0; n < RB; ++n) {
              float* r0 = &mine[m * 16 + g][n * 8 + 2 * c];
              float* r1 = &mine[m * 16 + g + 8][n * 8 + 2 * c];
              if (round == 0) { r0[0] = acc[m][n][0]; r0[1] = acc[m][n][1]; r1[0] = acc[m][n][2]; r1[1] = acc[m][n][3]; }
              else { r0[0] += acc[m][n][0]; r0[1] += acc[m][n][1]; r1[0] += acc[m][n][2]; r1[1] += acc[m][n][3]; }
              acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");    // consumers only
      }
      const int c0 = (this_item * KC) / sa.units_per_cta, c1 = (this_item * KC + KC - 1) / sa.units_per_cta;
      bool finish = true;                // does this CTA write the item's final result?
      if (c0 != c1) {
        const int slot = (this_item == (cta * sa.units_per_cta) / KC) ? 0 : 1;
        float* mine = a.partial + ((size_t)cta * 2 + slot) * (32 * R);
        for (int idx = threadIdx.x; idx < cur_nrows * R; idx += STREAM_WARPS * 32) {
          const int r = idx / R, q = idx % R;
          float v = 0.f;
#pragma unroll
          for (int w = 0; w < RW; ++w) v += red[w][r][q];
          mine[idx] = v;
        }
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");
        if (threadIdx.x == 0) is_last = (atomicAdd(a.counters + this_item, 1) == c1 - c0);
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");
        finish = is_last != 0;
        if (finish) __threadfence();
      }
      if (finish) {
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int idx = (int)threadIdx.x + k * STREAM_WARPS * 32;
          const int r = idx / R, q = idx % R;
          if (r >= cur_nrows) continue;
          float v = 0.f;
          if (c0 != c1) {
            for (int cc = c0; cc <= c1; ++cc) {        // fixed order: by CTA index
              const int slot = (this_item == (cc * sa.units_per_cta) / KC) ? 0 : 1;
              v += __ldcg(a.partial + ((size_t)cc * 2 + slot) * (32 * R) + idx);
            }
          } else {
#pragma unroll
            for (int w = 0; w < RW; ++w) v += red[w][r][q];
          }
          if (DROP && my_save[k] >= 0) v *= sa.drop.keep_scale;
          const float vs = v * my_scale;
          a.Out[(size_t)my_row[k] * R + q] = vs;
          fin[r][q] = vs;
          if (my_save[k] >= 0 && a.u_save) a.u_save[(size_t)(a.save_base + my_save[k]) * R + q] = v;
        }
        if (c0 != c1 && threadIdx.x == 0) a.counters[this_item] = 0;    // ready for the next launch
        if (a.pbd.pbd) {
          asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");  // fin[] complete
#pragma unroll
          for (int j = 0; j < 32 / STREAM_WARPS; ++j)
            if (pb_row[j] >= 0)
              pbd_write_row_at<R>(a.pbd, pb_row[j], pb_goff[j], pb_G[j], pb_g[j], fin[warp + STREAM_WARPS * j], pb_scale, lane);
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");      // red[] and fin[] are reused by the next item
    }
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
  DropArgs drop = {0, 0, 1.0f}; // per-item kernel with DROP (dA): elements of Q kept or dropped, P counts keep_scale
};

// grid = (D / 64, n_slots, ceil(R / (16 MB))).  A CTA owns a 64-column strip of one slot's
// gradient (and MB blocks of 16 rank rows); its 8 warps share the slot's row chunks, each
// accumulating G^T-style with the rows as the MMA's contraction index, and are summed in a fixed
// order, so the result does not depend on scheduling.  P is split into a bf16 head and a bf16
// remainder (two MMAs) to keep ~16 bits of its mantissa.
template <int MB, bool DROP = false>
__global__ void __launch_bounds__(GRAD_THREADS, MB == 1 ? 2 : 1)
grad_kernel(const GradArgs a) {
  extern __shared__ float grad_smem[];
  float (*red)[MB * 16][64 + 1] = reinterpret_cast<float (*)[MB * 16][64 + 1]>(grad_smem);
  const int slot = blockIdx.y;
  const int j0 = blockIdx.x * 64;
  const int qbase = blockIdx.z * MB * 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const int slot_ad = a.slot_adapter[slot];
  const int R = a.R;

  float acc[MB][8][4];
#pragma unroll
  for (int m = 0; m < MB; ++m)
#pragma unroll
    for (int n = 0; n < 8; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;

  const int ch0 = a.slot_chunk_off[slot], ch1 = a.slot_chunk_off[slot + 1];
  ptx::grid_dependency_wait();       // only plan tables were read so far
  ptx::grid_launch_dependents();
  const float sc = (a.scale ? a.scale[slot_ad] : 1.0f) * (DROP ? a.drop.keep_scale : 1.0f);
  const uint4 zero4 = make_uint4(0, 0, 0, 0);
  const int tr[4] = {2 * c, 2 * c + 1, 2 * c + 8, 2 * c + 9};
  // Two-deep register pipeline: the loads of chunk i+1 (4 rows of Q, 8 values of P per rank
  // block) are issued before the MMAs of chunk i.
  struct ChunkRegs { uint4 q[4]; float pv[MB][4][2]; };
  auto load_chunk = [&](int ch, ChunkRegs& r) {
    const int row0 = a.chunk_row0[ch], nrows = a.chunk_nrows[ch];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      r.q[i] = tr[i] < nrows ? ptx::ldg_nc_v4(a.Q + (size_t)(row0 + tr[i]) * a.ldq + j0 + 8 * g) : zero4;
      if (DROP && tr[i] < nrows) drop_mask8(a.drop, (uint32_t)(row0 + tr[i]), (uint32_t)(j0 + 8 * g), r.q[i]);   // compact row = place in save order
    }
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

// ---------------------------------------------------------------------------------------------
// Streaming gradient kernel for ranks up to 32.  A persistent CTA takes whole (slot, 512-column
// strip) groups in turn; for each it streams the slot's rows as tiles of 64 rows x 512 columns
// (ONE tensor-map load: eight 64-column blocks of [64 rows][128 B], 128B-swizzled, i.e. 1 KiB
// contiguous per row in memory) together with the matching 64 x R block of P (one bulk copy)
// through a ring of three stages.  Consumer warp w owns column block w of the strip for the whole
// group: it contracts all rows of every tile (four MMA K-steps, rows as the contraction index)
// into its own 16 (or 32) x 64 accumulator, so no reduction across warps is needed and the result
// goes from registers to memory; rows are visited in one fixed order, so the sums are
// run-to-run bit-reproducible.  The consumers read no table: the producer leaves each tile's row
// count in shared memory beside the tile.
// Narrow problems (few slots x strips for the SMs there are) use 256-column strips instead: four
// column blocks, and the two warps of a column block take the upper and the lower half of every
// tile's rows; the lower-half warps hand their accumulators over through shared memory at the end
// of the group (one fixed order again).
constexpr int GW_ROWS = 64;           // rows per staged tile
__host__ __device__ constexpr int gw_stages(int cb, int mb) {
  return mb >= 4 ? (cb == 8 ? 2 : 3) : (cb == 8 ? 3 : (mb == 1 ? 5 : 4));     // what fits 227 KiB of shared memory
}
__host__ __device__ constexpr size_t gw_smem_bytes(int cb, int mb) {
  return (size_t)gw_stages(cb, mb) * ((size_t)cb * GW_ROWS * 128 + (size_t)GW_ROWS * mb * 16 * 4) +
         (cb == 8 ? 0 : (size_t)cb * mb * 16 * 65 * 4) + 1024;
}

// One launch computes both gradients of a backward: problem 0 (dB: P = u_save scaled, Q = dY,
// D = d_out) and problem 1 (dA: P = V, Q = x_save, D = d_in); groups of problem 0 come first.
struct GradProblem {
  const float* P;              // [rows, R] fp32
  const float* scale;          // nullable
  float* G;                    // [n_slots, R, D]
  int32_t D, n_strips;         // ceil(D / strip width)
  DropArgs drop;               // dA with dropout: Q elements kept or dropped, P counts keep_scale (thr == 0: off)
};
struct GradStreamArgs {
  GradProblem prob[2];
  int32_t n_problems;          // 1 or 2
  int32_t R, accumulate;
  const int32_t* slot_adapter;
  const int32_t* slot_blk_off;
  const int32_t* blk_row0;     // blocks of <= 128 rows of one slot (compact fine-tuning rows)
  const int32_t* blk_nrows;
  int32_t n_slots;
  int32_t* status;
  // Few groups for the SMs there are (one or two fine-tuning adapters): the row blocks of a slot are
  // dealt out over n_parts CTAs per group; each leaves its fp32 sums in part_ws[group * n_parts +
  // part][16 MB][strip width], and the CTA that arrives last at part_counters[group] adds the parts
  // in index order (so the result does not depend on who was last) and writes the gradient.
  int32_t n_parts;             // >= 1
  float* part_ws;
  int32_t* part_counters;      // [groups], zero between launches
};

template <int MB, bool DROP, int CB>
__global__ void __launch_bounds__(STREAM_THREADS, 1)
grad_stream_kernel(const __grid_constant__ CUtensorMap tmQ0, const __grid_constant__ CUtensorMap tmQ1,
                   const GradStreamArgs ga) {
  static_assert(CB == 8 || CB == 4, "column blocks per strip");
  constexpr int S = gw_stages(CB, MB);
  constexpr int RMAX = MB * 16;
  constexpr int RH = STREAM_WARPS / CB;                  // warps sharing a column block (row halves of a tile)
  constexpr int KS_PER_WARP = (GW_ROWS / 16) / RH;
  constexpr int GW_COLS = CB * 64;
  constexpr uint32_t GW_Q_BYTES = CB * GW_ROWS * 128;
  constexpr uint32_t P_BYTES = GW_ROWS * RMAX * 4;
  constexpr uint32_t STAGE_BYTES = GW_Q_BYTES + P_BYTES;
  extern __shared__ __align__(1024) uint8_t gs_smem[];
  __shared__ __align__(8) uint64_t bars[2 * S];
  __shared__ int stage_meta[S][2];     // {first compact row, rows | last-tile-of-group flag << 16} of the staged tile
  __shared__ int abort_word;
  __shared__ int part_is_last;
  volatile int* abort_flag = &abort_word;
  const int R = ga.R;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (ptx::smem_u32(gs_smem) + 1023u) & ~1023u;      // swizzled tiles need 1 KiB alignment
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto bar_full = [&](int st) { return bar0 + 8u * st; };
  auto bar_empty = [&](int st) { return bar0 + 8u * (S + st); };
  // hand-over buffer of the lower-half warps (CB == 4 only), after the ring
  float (*red)[MB * 16][64 + 1] = reinterpret_cast<float (*)[MB * 16][64 + 1]>(
      gs_smem + (ring - ptx::smem_u32(gs_smem)) + S * STAGE_BYTES);
  if (threadIdx.x == 0) {
    for (int st = 0; st < S; ++st) { ptx::mbar_init(bar_full(st), 1); ptx::mbar_init(bar_empty(st), STREAM_WARPS); }
    abort_word = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ0);
    ptx::prefetch_tmap(&tmQ1);
  }
  __syncthreads();
  const int groups0 = ga.n_slots * ga.prob[0].n_strips;
  const int n_groups = groups0 + (ga.n_problems > 1 ? ga.n_slots * ga.prob[1].n_strips : 0);
  const int NP = ga.n_parts;
  const int n_units = n_groups * NP;       // unit = group * NP + part

  if (warp == STREAM_WARPS) {
    // ======================= producer =======================
    // the plan's tables are not written by the kernel before this one: the first group's entries
    // are fetched while that kernel may still be running
    // the blocks [b0, b1) of a slot's blocks [s_begin, s_end) that part `part` of NP takes
    auto part_range = [&](int s_begin, int s_end, int part, int& b0, int& b1) {
      const int per = (s_end - s_begin + NP - 1) / NP;
      b0 = min(s_end, s_begin + part * per);
      b1 = min(s_end, b0 + per);
    };
    int first_b_begin = 0, first_b_end = 0, first_row0 = 0, first_nrows = 0;
    if (lane == 0 && (int)blockIdx.x < n_units) {
      const int grp0 = (int)blockIdx.x / NP;
      const int pi = grp0 >= groups0 ? 1 : 0;
      const int slot = (grp0 - pi * groups0) / ga.prob[pi].n_strips;
      part_range(ga.slot_blk_off[slot], ga.slot_blk_off[slot + 1], (int)blockIdx.x % NP, first_b_begin, first_b_end);
      if (first_b_begin < first_b_end) { first_row0 = ga.blk_row0[first_b_begin]; first_nrows = ga.blk_nrows[first_b_begin]; }
    }
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    if (lane == 0) {
      uint32_t i = 0;
      bool ok = true;
      for (int un = blockIdx.x; un < n_units && ok; un += gridDim.x) {
        const int grp = un / NP;
        const int pi = grp >= groups0 ? 1 : 0;
        const GradProblem& pr = ga.prob[pi];
        const CUtensorMap* tmQ = pi ? &tmQ1 : &tmQ0;
        const int gl = grp - pi * groups0;
        const int slot = gl / pr.n_strips, strip = gl % pr.n_strips;
        const bool first = un == (int)blockIdx.x;
        int b_begin = first_b_begin, b_end = first_b_end;
        if (!first) part_range(ga.slot_blk_off[slot], ga.slot_blk_off[slot + 1], un % NP, b_begin, b_end);
        if (b_begin == b_end) {            // no rows (an empty slot, or a part past the slot's blocks): an empty last tile, so that the sums are still written
          const int st = i % S;
          if (!(ok = stream_wait(bar_empty(st), ((i / S) & 1) ^ 1, abort_flag, ga.status))) break;
          stage_meta[st][0] = 0;
          stage_meta[st][1] = 1 << 16;
          ptx::mbar_arrive(bar_full(st));
          ++i;
          continue;
        }
        int row0 = first ? first_row0 : ga.blk_row0[b_begin], nrows = first ? first_nrows : ga.blk_nrows[b_begin];
        for (int b = b_begin; b < b_end && ok; ++b) {
          // the next block's table entries are requested before this block's tiles are waited for
          const int nb1 = b + 1 < b_end ? b + 1 : b;
          const int next_row0 = ga.blk_row0[nb1], next_nrows = ga.blk_nrows[nb1];
          for (int off = 0; off < nrows; off += GW_ROWS, ++i) {
            const int st = i % S;
            if (!(ok = stream_wait(bar_empty(st), ((i / S) & 1) ^ 1, abort_flag, ga.status))) break;
            const int nr = min(GW_ROWS, nrows - off);
            const uint32_t dst = ring + (uint32_t)st * STAGE_BYTES;
            const uint32_t pbytes = (uint32_t)nr * (uint32_t)R * 4u;
            stage_meta[st][0] = row0 + off;
            stage_meta[st][1] = nr | ((b == b_end - 1 && off + GW_ROWS >= nrows) ? (1 << 16) : 0);
            ptx::mbar_arrive_expect_tx(bar_full(st), GW_Q_BYTES + pbytes);
            // rows past the tile's count are masked by the consumers; blocks past D arrive as zeros
            ptx::tma_load_3d(dst, tmQ, 0, row0 + off, strip * CB, bar_full(st));
            bulk_load(dst + GW_Q_BYTES, pr.P + (size_t)(row0 + off) * R, pbytes, bar_full(st));
          }
          row0 = next_row0; nrows = next_nrows;
        }
      }
    }
  } else {
    // ======================= consumers =======================
    const int g = lane >> 2, c = lane & 3;
    ptx::grid_dependency_wait();
    float acc[MB][8][4];
    uint32_t i = 0;
    bool ok = true;
    for (int un = blockIdx.x; un < n_units && ok; un += gridDim.x) {
      const int grp = un / NP;
      const int pi = grp >= groups0 ? 1 : 0;
      const GradProblem& pr = ga.prob[pi];
      const int gl = grp - pi * groups0;
      const int slot = gl / pr.n_strips, strip = gl % pr.n_strips;
      const int cblk = warp % CB, half = warp / CB;
      const int col0 = strip * GW_COLS + cblk * 64;        // this warp's 64 columns
      const bool active = col0 < pr.D;
      const float sc = (pr.scale ? pr.scale[ga.slot_adapter[slot]] : 1.0f) * ((DROP && pr.drop.thr != 0) ? pr.drop.keep_scale : 1.0f);
#pragma unroll
      for (int m = 0; m < MB; ++m)
#pragma unroll
        for (int n = 0; n < 8; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;
      for (bool last = false; !last; ++i) {
        const int st = i % S;
        if (!(ok = stream_wait(bar_full(st), (i / S) & 1, abort_flag, ga.status))) break;
        const int trow0 = stage_meta[st][0];
        const int meta = stage_meta[st][1];
        const int nrows = meta & 0xFFFF;
        last = (meta >> 16) != 0;
        // plain shared-memory loads (no branches around them): what lies past a tile's rows is read
        // and then replaced by zero
        const uint8_t* stage_ptr = gs_smem + (ring - ptx::smem_u32(gs_smem)) + (size_t)st * STAGE_BYTES;
        const uint8_t* qtile = stage_ptr + (size_t)cblk * (GW_ROWS * 128u);
        const float* ptile = reinterpret_cast<const float*>(stage_ptr + GW_Q_BYTES);
        if (active) {
#pragma unroll
          for (int kk = 0; kk < KS_PER_WARP; ++kk) {
            const int ks = half * KS_PER_WARP + kk;
            if (ks * 16 >= nrows) break;
            // rows of this K-step: r = 16 ks + {2c, 2c+1, 2c+8, 2c+9}
            uint4 q[4];
            uint32_t ahi[MB][4], alo[MB][4];
            const int tr[4] = {2 * c, 2 * c + 1, 2 * c + 8, 2 * c + 9};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int r = ks * 16 + tr[k];
              // 16-byte piece g of row r sits at piece (g ^ (r & 7)) of the swizzled 128-byte row
              const uint4 t = *reinterpret_cast<const uint4*>(qtile + r * 128 + ((g ^ (r & 7)) << 4));
              const bool in = r < nrows;                           // rows of the tile past the block's end count zero
              q[k] = make_uint4(in ? t.x : 0u, in ? t.y : 0u, in ? t.z : 0u, in ? t.w : 0u);
              if (DROP && in && pr.drop.thr != 0) drop_mask8(pr.drop, (uint32_t)(trow0 + r), (uint32_t)(col0 + 8 * g), q[k]);
            }
#pragma unroll
            for (int m = 0; m < MB; ++m) {
              float pv[4][2];
#pragma unroll
              for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                  const int r = ks * 16 + tr[k], qq = m * 16 + g + 8 * h;
                  const float v = ptile[r * R + qq];               // inside the stage's P area for every r < 64, qq < 16 MB
                  pv[k][h] = (r < nrows && qq < R) ? v * sc : 0.f;
                }
#pragma unroll
              for (int f = 0; f < 4; ++f) {       // a0 (q=g, rows 2c,2c+1), a1 (q=g+8, same rows), a2, a3: rows 2c+8,2c+9
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
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_empty(st));
      }
      if (!ok) break;
      // ---- group done: this warp's 16 (32) x 64 block goes from registers to the gradient ----
      // The n index g of the MMA was mapped to piece g of a row, so for thread (g, c) accumulator
      // element e of column block nb is strip column 8 (2c + (e & 1)) + nb: over nb = 0..7 that is
      // eight consecutive columns, written as two 16-byte stores (rows g and g + 8 for e >> 1).
      if (RH == 2) {       // the lower-half warp of a column block hands its sums to the upper-half warp
        if (half == 1) {
#pragma unroll
          for (int m = 0; m < MB; ++m)
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
              for (int e = 0; e < 4; ++e)
                red[cblk][m * 16 + g + ((e >> 1) ? 8 : 0)][8 * (2 * c + (e & 1)) + nb] = acc[m][nb][e];
        }
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");
        if (half == 0) {
#pragma unroll
          for (int m = 0; m < MB; ++m)
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
              for (int e = 0; e < 4; ++e)
                acc[m][nb][e] += red[cblk][m * 16 + g + ((e >> 1) ? 8 : 0)][8 * (2 * c + (e & 1)) + nb];
        }
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");   // red[] is reused by the next group
      }
      bool write_out = true;
      if (NP > 1) {        // row-split group: leave this part's sums, the last arrival adds all parts in index order
        if (active && half == 0) {
          float* mine = ga.part_ws + (size_t)un * (RMAX * GW_COLS);
#pragma unroll
          for (int m = 0; m < MB; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int ql = m * 16 + g + ((e >> 1) ? 8 : 0);
              float4* dst = reinterpret_cast<float4*>(mine + (size_t)ql * GW_COLS + cblk * 64 + 8 * (2 * c + (e & 1)));
              dst[0] = make_float4(acc[m][0][e], acc[m][1][e], acc[m][2][e], acc[m][3][e]);
              dst[1] = make_float4(acc[m][4][e], acc[m][5][e], acc[m][6][e], acc[m][7][e]);
            }
        }
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");
        if (threadIdx.x == 0) part_is_last = (atomicAdd(ga.part_counters + grp, 1) == NP - 1);
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");
        write_out = part_is_last != 0;
        if (write_out) {
          __threadfence();
          if (active && half == 0) {
#pragma unroll
            for (int m = 0; m < MB; ++m)
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int ql = m * 16 + g + ((e >> 1) ? 8 : 0);
                float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
                for (int pp = 0; pp < NP; ++pp) {
                  const float4* src = reinterpret_cast<const float4*>(
                      ga.part_ws + ((size_t)grp * NP + pp) * (RMAX * GW_COLS) + (size_t)ql * GW_COLS + cblk * 64 + 8 * (2 * c + (e & 1)));
                  const float4 a0 = __ldcg(src), a1 = __ldcg(src + 1);
                  lo.x += a0.x; lo.y += a0.y; lo.z += a0.z; lo.w += a0.w;
                  hi.x += a1.x; hi.y += a1.y; hi.z += a1.z; hi.w += a1.w;
                }
                acc[m][0][e] = lo.x; acc[m][1][e] = lo.y; acc[m][2][e] = lo.z; acc[m][3][e] = lo.w;
                acc[m][4][e] = hi.x; acc[m][5][e] = hi.y; acc[m][6][e] = hi.z; acc[m][7][e] = hi.w;
              }
          }
          if (threadIdx.x == 0) ga.part_counters[grp] = 0;       // ready for the next launch
        }
        asm volatile("bar.sync 1, %0;" ::"n"(STREAM_WARPS * 32) : "memory");   // part_is_last is reused by the next group
      }
      if (write_out && active && half == 0) {
#pragma unroll
        for (int m = 0; m < MB; ++m)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int ql = m * 16 + g + ((e >> 1) ? 8 : 0);
            if (ql >= R) continue;
            float4* dst = reinterpret_cast<float4*>(pr.G + ((size_t)slot * R + ql) * pr.D + col0 + 8 * (2 * c + (e & 1)));
            float4 lo = make_float4(acc[m][0][e], acc[m][1][e], acc[m][2][e], acc[m][3][e]);
            float4 hi = make_float4(acc[m][4][e], acc[m][5][e], acc[m][6][e], acc[m][7][e]);
            if (ga.accumulate) {
              const float4 o0 = dst[0], o1 = dst[1];
              lo.x += o0.x; lo.y += o0.y; lo.z += o0.z; lo.w += o0.w;
              hi.x += o1.x; hi.y += o1.y; hi.z += o1.z; hi.w += o1.w;
            }
            dst[0] = lo;
            dst[1] = hi;
          }
      }
    }
  }
}

// Low-rank part of the input gradient under dropout: dX[m, k] += keep(m, k) / (1 - p) *
// sum_q V[m, q] A_a(m)[q, k].
struct ExpandMaskArgs {
  const float* V;                 // [rows, R] fp32 (already scaled by s)
  int32_t R;
  const __nv_bfloat16* A_all;     // [n_adapters, R, D]
  const int32_t* row_adapter;     // [rows] over the compact fine-tuning rows
  __nv_bfloat16* dX;              // [rows, D], row stride lddx
  int64_t lddx;
  int32_t D, n_rows;
  DropArgs drop;
};

constexpr int EM_ROWS = 8;       // rows per block of the masked expand

// grid = (ceil(rows / EM_ROWS), column blocks of 128 x 8); one thread per 8 columns and EM_ROWS rows.
// Rows of a block that share their adapter (the usual case: fine-tuning rows of one sequence) read each
// piece of A once for all of them; a block with mixed adapters takes its rows one by one.
__global__ void __launch_bounds__(128)
expand_mask_kernel(const ExpandMaskArgs a) {
  __shared__ float v[EM_ROWS][kMaxRank];
  __shared__ int ads[EM_ROWS];
  const int m0 = blockIdx.x * EM_ROWS;
  const int k = (blockIdx.y * 128 + threadIdx.x) * 8;
  if (threadIdx.x < EM_ROWS) ads[threadIdx.x] = (m0 + (int)threadIdx.x < a.n_rows) ? a.row_adapter[m0 + threadIdx.x] : -1;
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  for (int idx = threadIdx.x; idx < EM_ROWS * a.R; idx += 128) {
    const int r = idx / a.R, q = idx % a.R;
    v[r][q] = (m0 + r < a.n_rows) ? a.V[(size_t)(m0 + r) * a.R + q] : 0.f;
  }
  __syncthreads();
  if (k >= a.D) return;
  bool same = true;
#pragma unroll
  for (int r = 1; r < EM_ROWS; ++r) same = same && (ads[r] == ads[0] || ads[r] < 0);
  float acc[EM_ROWS][8];
#pragma unroll
  for (int r = 0; r < EM_ROWS; ++r)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[r][i] = 0.f;
  if (same && ads[0] >= 0) {
    const __nv_bfloat16* Ab = a.A_all + (size_t)ads[0] * a.R * a.D + k;
    for (int q = 0; q < a.R; ++q) {
      const uint4 w = ptx::ldg_nc_v4(Ab + (size_t)q * a.D);
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int r = 0; r < EM_ROWS; ++r) {
        const float vq = v[r][q];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[r][2 * i] = fmaf(vq, __uint_as_float(ww[i] << 16), acc[r][2 * i]);
          acc[r][2 * i + 1] = fmaf(vq, __uint_as_float(ww[i] & 0xFFFF0000u), acc[r][2 * i + 1]);
        }
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < EM_ROWS; ++r) {
      if (ads[r] < 0) continue;
      const __nv_bfloat16* Ab = a.A_all + (size_t)ads[r] * a.R * a.D + k;
      for (int q = 0; q < a.R; ++q) {
        const uint4 w = ptx::ldg_nc_v4(Ab + (size_t)q * a.D);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
        const float vq = v[r][q];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[r][2 * i] = fmaf(vq, __uint_as_float(ww[i] << 16), acc[r][2 * i]);
          acc[r][2 * i + 1] = fmaf(vq, __uint_as_float(ww[i] & 0xFFFF0000u), acc[r][2 * i + 1]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < EM_ROWS; ++r) {
    const int m = m0 + r;
    if (ads[r] < 0) continue;               // also rows past the end
    const uint64_t z0 = drop_bits(a.drop.seed, (uint32_t)m, (uint32_t)(k >> 2));
    const uint64_t z1 = drop_bits(a.drop.seed, (uint32_t)m, (uint32_t)(k >> 2) + 1);
    __nv_bfloat16* dst = a.dX + (size_t)m * a.lddx + k;
    const uint4 o = *reinterpret_cast<const uint4*>(dst);
    uint32_t ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint64_t z = i < 2 ? z0 : z1;
      const int f = (2 * i) & 3;
      const bool k0 = (uint32_t)((z >> (16 * f)) & 0xFFFFu) >= a.drop.thr;
      const bool k1 = (uint32_t)((z >> (16 * (f + 1))) & 0xFFFFu) >= a.drop.thr;
      const float lo = __uint_as_float(ow[i] << 16) + (k0 ? acc[r][2 * i] * a.drop.keep_scale : 0.f);
      const float hi = __uint_as_float(ow[i] & 0xFFFF0000u) + (k1 ? acc[r][2 * i + 1] * a.drop.keep_scale : 0.f);
      ow[i] = ptx::pack_bf16(lo, hi);
    }
    *reinterpret_cast<uint4*>(dst) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
  }
}

}  // namespace mlora
