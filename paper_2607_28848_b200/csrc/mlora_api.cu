// C ABI of the mixed-batch multi-LoRA layer: context, plan upload, argument checks, tensor-map
// encoding and kernel dispatch.  See include/mlora.h for the contract of every entry point.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <algorithm>
#include <mutex>
#include <queue>
#include <new>
#include <utility>
#include <vector>

#include "mlora.h"
#include "plan.h"
#include "gemm_tcgen05.cuh"
#include "gemm2_tcgen05.cuh"
#include "simt.cuh"
#include "skinny.cuh"
#include "grad_tc.cuh"
#include "shrink_tc.cuh"
#include "glue.cuh"
#include "attention.cuh"
#include "attention_tc.cuh"
#include "mlora_layer_ops.h"

using namespace mlora;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Device tables + pinned staging of a stream-ordered plan; `free_evt` marks the point on a stream
// after which the pair may be reused.
struct PlanBuf {
  int32_t* dev = nullptr;
  int32_t* pinned = nullptr;
  size_t cap = 0;                    // in 32-bit words
  cudaEvent_t free_evt = nullptr;
};
static inline void free_plan_buf(PlanBuf& b) {
  if (b.dev) cudaFree(b.dev);
  if (b.pinned) cudaFreeHost(b.pinned);
  if (b.free_evt) cudaEventDestroy(b.free_evt);
  b = PlanBuf();
}

struct mlora_ctx {
  int device = 0;
  int sm_count = 0;
  int32_t* status_dev = nullptr;     // device status word
  float* ws_p = nullptr;             // [ws_rows, kMaxRank] rank-r intermediate of the running call
  int64_t ws_rows = 0;
  float* ws_partial = nullptr;       // split-K partials of the shrink kernel: [ws_partial_items, 32, kMaxRank]
  int64_t ws_partial_items = 0;
  int32_t* ws_counters = nullptr;    // [ws_counter_items] arrival counters, zero between launches
  int64_t ws_counter_items = 0;
  __nv_bfloat16* ws_pbd = nullptr;   // block-diagonal low-rank operand: [2 * ws_pbd_groups * 256, 64] bf16
  int64_t ws_pbd_groups = 0;
  float* ws_splitk = nullptr;        // fp32 partial products of a K-split GEMM (fixed size, see kSplitKBytes)
  float* ws_gpart = nullptr;         // partial gradient sums that several CTAs share: [sm_count][4][64 KiB] (the streaming kernel's
                                     // row-split groups use the first 128 KiB per SM, the tensor-core kernel's split strips all of it)
  int32_t* ws_gcounters = nullptr;   // [sm_count] arrival counters of those groups, zero between launches
  uint8_t* ws_pop = nullptr;         // P operands of the tensor-core gradient kernel: [2][ws_pop_blocks][64 KiB]
  int64_t ws_pop_blocks = 0;
  float* ws_tc_part = nullptr;       // run sums of the tensor-core shrink: [ws_rows + 128 * sm_count][kMaxRank]
  int32_t* ws_tc_counters = nullptr; // [kTcCounters] counters of the tensor-core gradient kernel, zero between launches
  std::vector<void*> retired;        // workspaces replaced by larger ones: kept until the context is destroyed,
                                     // because a captured graph may still hold their addresses
  std::vector<PlanBuf> plan_pool;    // released buffers of stream-ordered plans
  int64_t launches = 0;
  int32_t gemm_path = 0;
  int32_t shrink_path = 0;           // 0: default choice by rank (streaming mma.sync kernels, tcgen05 kernels from rank 64); 1: per-item kernels for every rank
  int32_t gemm_pairs = 1;            // 1: two-SM (CTA pair) tensor-core kernel; 0: one-SM kernel
  int32_t no_split_k = 0;            // 1: the two-SM kernel never splits K (kernel variant 4)
  int32_t no_unit_lists = 0;         // 1: the two-SM kernel always deals its units out round robin (kernel variant 7)
  int32_t grad_mode = 0;             // 0: default choice by rank; 1: mma.sync kernels for every rank (kernel variant 5);
                                     // 2: the tcgen05 shrink and gradient kernels for every rank (kernel variant 6)
  EncodeTiledFn encode = nullptr;
  const volatile int32_t* cancel = nullptr;   // caller's host flag, read before every launch
  DropArgs drop = {0, 0, 1.0f};               // LoRA dropout of the fine-tuning rows (thr == 0: off)
  // optional per-launch timing
  std::vector<cudaEvent_t> ev_start, ev_stop;
  std::vector<int32_t> ev_kind;
  int32_t ev_used = 0;
};

constexpr int kMaxKSplit = 16;
// Ranks from which the tcgen05 gradient kernel (with its P operands made ahead by psplit_kernel) is the default.
// Measured on B200 (both launches with their event pairs, 4096 -> 14336, 1024 fine-tuning rows), against the mma.sync
// streaming kernel: rank 16 7 + 27 vs 21 us, rank 32 8 + 23 vs 29, rank 64 9 + 25 vs 33-50 (whole step 295 vs 315 us with
// one adapter, 404 vs 410 with 256), rank 128 9 + 25 vs 144 (two launches of the per-item kernel).  Before the operands
// were made ahead, every tile converted its own (rank 128: 7 us per tile, 56-70 us per launch).  Rank 32 is a draw launch by
// launch and 2% ahead in the step where the fine-tuning rows come in long runs (5120 -> 13824, 2048 fine-tuning rows of one
// adapter, forward + backward with both tcgen05 families: 448 vs 458 us; with 512 decode rows beside them 575 vs 587).
constexpr int kTcGradMinRank = 32;
// Ranks from which the tcgen05 shrink (U = X A^T with the activation save, V = s dY B^T) is the default.  Measured on
// B200 (main + finish launch with their event pairs, 2048 x 4096 forward / 1024 x 14336 backward): rank 128 19 + 12 and
// 20 + 10 us vs 43 and 74 for the per-item kernel; rank 64 15 + 13 and 17 + 9 vs 31 and 37 for the streaming kernel;
// rank 32 14 + 15 and 17 + 9 vs 20 and 25 one by one, but inside the step (launch overlap on) the pair is the faster one
// (see above), hence the default from rank 32.
constexpr int kTcShrinkMinRank = 32;

enum { KIND_SHRINK = 0, KIND_GEMM_FWD = 1, KIND_GEMM_BWD = 2, KIND_GRAD = 3, KIND_SIMT = 4, KIND_ADAMW = 5, KIND_REDUCE = 6 };

// Cost-balanced unit lists of the two-SM GEMM (see balanced_units), cached per plan and row space: a
// batch whose row tiles differ much in their number of adapter groups gets, per (columns, depth, rank)
// it is used with, one list in device memory reserved with the plan's tables.
constexpr int kSchedSlots = 4;          // shapes per row space; further shapes run round robin
constexpr int kSchedCap = 8192;         // 32-bit words per list (pairs + 1 offsets, then the units)
struct SchedEntry {
  int32_t n_ntiles = 0, kblocks = 0, rank = 0, pairs = 0, n_whole = 0, n_tail = 0, split_k = 0, group_m = 0;
  bool use = false;                     // false: round robin is as good for this shape
  cudaEvent_t filled = nullptr;         // recorded behind the copy that fills the device list
  cudaStream_t stream = nullptr;        // the stream of that copy
};
struct SchedCache {
  std::mutex mu;
  int32_t* dev = nullptr;               // [kSchedSlots][kSchedCap], nullptr: nothing reserved (even row space)
  int32_t* mirror = nullptr;            // the same area in pinned host memory: source of the copies (a copy from
                                        // pageable memory would make the runtime wait for the stream first)
  int32_t n = 0;
  int32_t lc_spread = 0;                // most minus fewest adapter groups of a 256-row tile
  SchedEntry e[kSchedSlots];
  ~SchedCache() { for (SchedEntry& x : e) if (x.filled) cudaEventDestroy(x.filled); }
};

// Device copy of one RowSpace.
struct DevRowSpace {
  SchedCache* sched = nullptr;
  const int32_t* row_adapter = nullptr;
  const int32_t* row_save = nullptr;
  const int32_t* row_grp = nullptr;
  const int32_t* tile_grp_off = nullptr;
  const int32_t* grp_adapter = nullptr;
  const int32_t* row_grp2 = nullptr;
  const int32_t* tile2_grp_off = nullptr;
  const int32_t* grp2_adapter = nullptr;
  const int32_t* zero_rows2 = nullptr;
  const int32_t* item_rows = nullptr;
  const int32_t* item_save = nullptr;
  const int32_t* item_start = nullptr;
  const int32_t* item_nrows = nullptr;
  const int32_t* item_adapter = nullptr;
  const int32_t* item_desc = nullptr;
  const int32_t* tcb_row0 = nullptr;
  const int32_t* tcb_nrows = nullptr;
  const int32_t* tcb_adapter = nullptr;
  const int32_t* tcb_width = nullptr;      // plans made with per-adapter ranks (null otherwise)
  // plans made with per-adapter ranks (null otherwise)
  const int32_t* grp2_col = nullptr;
  const int32_t* grp2_width = nullptr;
  const int32_t* tile2_cols = nullptr;
  const int32_t* tile2_piece_off = nullptr;
  const int32_t* piece_src = nullptr;
};

struct mlora_plan {
  HostPlan h;
  mlora_ctx* ctx = nullptr;
  int32_t* blob = nullptr;           // all device tables in one allocation
  PlanBuf buf;                       // pooled plans: the buffer pair the tables live in (blob == buf.dev)
  bool pooled = false;
  DevRowSpace fwd, bwd;
  SchedCache sched[2];               // unit lists of the forward and the compact row space
  int32_t* sched_pinned = nullptr;   // pinned mirror of the unit-list areas of a plan that is not pooled (every plan with a context is pooled now)
  const int32_t* slot_chunk_off = nullptr;
  const int32_t* chunk_row0 = nullptr;
  const int32_t* chunk_nrows = nullptr;
  const int32_t* slot_adapter = nullptr;
  const int32_t* slot_blk_off = nullptr;
  const int32_t* blk_row0 = nullptr;
  const int32_t* blk_nrows = nullptr;
  const int32_t* slot_width = nullptr;   // plans made with per-adapter ranks (null otherwise)
};

namespace {

struct BlobBuilder {
  std::vector<int32_t> data;
  size_t add(const std::vector<int32_t>& v) {
    const size_t off = data.size();
    data.insert(data.end(), v.begin(), v.end());
    while (data.size() % 4) data.push_back(0);      // keep every table 16-byte aligned
    if (v.empty()) { data.insert(data.end(), 4, 0); }
    return off;
  }
};

// Workspace for K-split products of small-batch GEMMs: allocated once per context, so that no
// compute call allocates.  Problems whose partials do not fit run unsplit.
constexpr size_t kSplitKBytes = 64u << 20;
constexpr int64_t kPopMaxBlocks = 512;  // most 128-row blocks whose gradient operands are made ahead (64 MiB)
constexpr int kTcCounters = 1 << 18;    // counter words of the tensor-core gradient kernel (1 MiB, allocated with the context)
constexpr int kMaxDevices = 64;      // device ordinals a process may create contexts on
// One-time kernel attributes (opt-in shared-memory size, resident cluster count) are cached per kernel
// instantiation and device in function-local arrays; contexts are independent across host threads, so
// two threads may reach the same cache at once: every read-check-set of such a cache holds this lock.
std::mutex g_attr_mutex;

// With MLORA_DEBUG set in the environment, the place and the runtime's message of a failed CUDA call go to stderr.
mlora_status_t cuda_failure(const char* site, const char* detail) {
  static const bool verbose = std::getenv("MLORA_DEBUG") != nullptr;
  if (verbose) std::fprintf(stderr, "mlora: CUDA failure at %s: %s\n", site, detail ? detail : "");
  return MLORA_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

mlora_status_t make_tmap_bf16(const mlora_ctx* ctx, CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer,
                              uint64_t row_stride_elems, uint32_t box_inner, uint32_t box_outer, bool swizzle = true) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_elems * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char msg[160];
    std::snprintf(msg, sizeof msg, "code %d, dims %llu x %llu, row stride %llu, box %u x %u, base %p", (int)r,
                  (unsigned long long)inner, (unsigned long long)outer, (unsigned long long)row_stride_elems, box_inner,
                  box_outer, base);
    return cuda_failure("tensor map (2-D)", msg);
  }
  return MLORA_OK;
}

// [rows, cols] (cols contiguous, a multiple of 64) seen as (64, rows, cols / 64): a box of
// 64 x box_rows x box_blocks lands in shared memory as box_blocks consecutive [box_rows][64]
// blocks, the MN-major operand layout of the tensor-core kernel.
mlora_status_t make_tmap_bf16_blocked(const mlora_ctx* ctx, CUtensorMap* m, const void* base, uint64_t rows,
                                      uint64_t cols, uint64_t row_stride_elems, uint32_t box_rows, uint32_t box_blocks) {
  cuuint64_t dims[3] = {64, rows, cols / 64};
  cuuint64_t strides[2] = {row_stride_elems * 2, 128};
  cuuint32_t box[3] = {64, box_rows, box_blocks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char msg[160];
    std::snprintf(msg, sizeof msg, "code %d, rows %llu, cols %llu, row stride %llu, box rows %u, blocks %u, base %p", (int)r,
                  (unsigned long long)rows, (unsigned long long)cols, (unsigned long long)row_stride_elems, box_rows,
                  box_blocks, base);
    return cuda_failure("tensor map (blocked)", msg);
  }
  return MLORA_OK;
}

bool rank_ok_bf16(int r) { return r == 8 || r == 16 || r == 32 || r == 64 || r == 128; }

mlora_status_t check_layer(const mlora_layer_t* L) {
  if (!L || !L->W || !L->A_all || !L->B_all || !L->scale) return MLORA_ERR_INVALID_ARG;
  if (L->d_in <= 0 || L->d_out <= 0 || L->rank <= 0 || L->n_adapters <= 0) return MLORA_ERR_INVALID_ARG;
  if (L->dtype != MLORA_F32 && L->dtype != MLORA_BF16) return MLORA_ERR_INVALID_ARG;
  if (L->ldw < L->d_out) return MLORA_ERR_INVALID_ARG;
  if (L->rank > kMaxRank) return MLORA_ERR_UNSUPPORTED;
  if (L->dtype == MLORA_BF16) {
    if (!rank_ok_bf16(L->rank) || L->d_in % 64 || L->d_out % 64 || L->ldw % 8) return MLORA_ERR_UNSUPPORTED;
    if (!aligned16(L->W) || !aligned16(L->A_all) || !aligned16(L->B_all)) return MLORA_ERR_UNSUPPORTED;
  }
  return MLORA_OK;
}

inline bool cancelled(const mlora_ctx* c) { return c->cancel && *c->cancel != 0; }

// Brackets one kernel launch: optional event pair, launch counter, launch-error check.
struct LaunchScope {
  mlora_ctx* ctx; cudaStream_t st; int slot;
  LaunchScope(mlora_ctx* c, cudaStream_t s, int kind) : ctx(c), st(s), slot(-1) {
    if (c->ev_used < (int32_t)c->ev_start.size()) {
      slot = c->ev_used++;
      c->ev_kind[slot] = kind;
      cudaEventRecord(c->ev_start[slot], st);
    }
  }
  mlora_status_t done() {
    if (slot >= 0) cudaEventRecord(ctx->ev_stop[slot], st);
    ctx->launches++;
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? MLORA_OK : cuda_failure("kernel launch", cudaGetErrorString(e));
  }
};

// Launch with programmatic stream serialization: the kernel may start its set-up while the
// previous kernel of the stream drains; it calls griddepcontrol.wait before touching data.
// Switched off while per-launch events are being recorded, so that those time whole kernels.
template <typename... KArgs, typename... Args>
void launch_pdl(bool overlap, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// Same, for a kernel whose CTAs come in clusters of two.
template <typename... KArgs, typename... Args>
void launch_pdl_pairs(bool overlap, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                      Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = 2; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// ---- bf16 launches ------------------------------------------------------------------------
template <int RB, int MT, int WARPS, int MIN_CTAS>
void launch_shrink_rb(bool overlap, const ShrinkArgs& a, int n_items, int ksplit, cudaStream_t st) {
  launch_pdl(overlap, shrink_kernel<RB, MT, WARPS, MIN_CTAS>, dim3(n_items, ksplit, kItemRows / (16 * MT)),
             dim3(WARPS * 32), 0, st, a);
}
// Few items with a long contraction leave most SMs idle: split K over several CTAs per item so
// that about three CTAs per SM are in flight, keeping at least 16 K-blocks (1024 elements) each.
int shrink_ksplit(const mlora_ctx* ctx, int n_items, int D) {
  const int want = (3 * ctx->sm_count + n_items - 1) / n_items;
  const int cap = D / 64 / 16;
  int k = want < cap ? want : cap;
  k = k < kMaxKSplit ? k : kMaxKSplit;
  return k < 1 ? 1 : k;
}
template <int RB, int STAGES, int CHUNK, bool DROP>
mlora_status_t launch_shrink_stream_d(mlora_ctx* ctx, ShrinkArgs a, int n_items, const int32_t* item_desc, int n_rows,
                                    int n_adapters, cudaStream_t st) {
  constexpr int R = RB * 8;
  constexpr size_t xrow = 32 * (CHUNK * 128 + 16), xtile = (size_t)(CHUNK / 4) * 32 * 512;
  constexpr size_t xbytes = ((xrow > xtile ? xrow : xtile) + 1023) / 1024 * 1024;
  constexpr size_t smem = 1024 + (size_t)STAGES * (xbytes + (size_t)(CHUNK / 4) * R * 512) +
                          (size_t)(RB >= 8 ? 2 : (RB >= 4 ? 4 : 8)) * 32 * (R + 1) * 4;
  CUtensorMap tIn, tP, tSave;
  mlora_status_t ms;
  // (64, rows, D / 64) views: one box = 4 K-blocks x rows x 128 bytes, 128-byte swizzle
  if ((ms = make_tmap_bf16_blocked(ctx, &tIn, a.In, n_rows, a.D, a.ld_in, 32, 4)) != MLORA_OK) return ms;
  if ((ms = make_tmap_bf16_blocked(ctx, &tP, a.P_all, (uint64_t)n_adapters * R, a.D, a.D, R, 4)) != MLORA_OK) return ms;
  // full items of fine-tuning rows are saved as blocks straight from the staged tiles
  const bool tma_save = a.x_save != nullptr && a.save_cap > 0;
  if (tma_save) {
    if ((ms = make_tmap_bf16_blocked(ctx, &tSave, a.x_save, (uint64_t)a.save_cap, a.D, a.D, 32, 4)) != MLORA_OK) return ms;
  } else {
    tSave = tIn;
  }
  static bool attr_set_dev[kMaxDevices] = {};   // per instantiation and device
  bool& attr_set = attr_set_dev[ctx->device];
  auto kern = shrink_stream_kernel<RB, STAGES, CHUNK, DROP>;
  {
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    if (!attr_set) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return MLORA_ERR_CUDA;
      attr_set = true;
    }
  }
  StreamArgs sa;
  sa.s = a;
  sa.s.partial = ctx->ws_partial;
  sa.s.counters = ctx->ws_counters;
  sa.n_items = n_items;
  sa.tma_save = tma_save ? 1 : 0;
  sa.drop = a.item_save ? ctx->drop : DropArgs{0, 0, 1.0f};   // only the forward's fine-tuning rows are dropped
  sa.chunks_per_item = (a.D / 64 + CHUNK - 1) / CHUNK;
  sa.n_units = n_items * sa.chunks_per_item;
  int grid = sa.n_units < ctx->sm_count ? sa.n_units : ctx->sm_count;
  sa.units_per_cta = (sa.n_units + grid - 1) / grid;
  grid = (sa.n_units + sa.units_per_cta - 1) / sa.units_per_cta;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  if (2 * (int64_t)grid > ctx->ws_partial_items || n_items > ctx->ws_counter_items) return MLORA_ERR_INVALID_ARG;
  LaunchScope scope(ctx, st, KIND_SHRINK);
  sa.status = ctx->status_dev;
  sa.item_desc = item_desc;
  launch_pdl(scope.slot < 0, kern, dim3(grid), dim3(STREAM_THREADS), smem, st, tIn, tP, tSave, sa);
  return scope.done();
}

// The dropout variant is its own instantiation, so that the usual one carries none of the mask arithmetic.
template <int RB, int STAGES, int CHUNK>
mlora_status_t launch_shrink_stream(mlora_ctx* ctx, ShrinkArgs a, int n_items, const int32_t* item_desc, int n_rows,
                                    int n_adapters, cudaStream_t st) {
  if constexpr (RB <= 8) {           // dropout is offered up to rank 64 (the streaming kernels' range)
    if (a.item_save && ctx->drop.thr != 0)
      return launch_shrink_stream_d<RB, STAGES, CHUNK, true>(ctx, a, n_items, item_desc, n_rows, n_adapters, st);
  }
  return launch_shrink_stream_d<RB, STAGES, CHUNK, false>(ctx, a, n_items, item_desc, n_rows, n_adapters, st);
}

mlora_status_t launch_shrink(mlora_ctx* ctx, int R, ShrinkArgs a, int n_items, const int32_t* item_desc, int n_rows,
                             int n_adapters, cudaStream_t st) {
  if (n_items <= 0) return MLORA_OK;
  if (ctx->shrink_path == 0) {
    if (R == 8) return launch_shrink_stream<1, 2, 16>(ctx, a, n_items, item_desc, n_rows, n_adapters, st);
    if (R == 16) return launch_shrink_stream<2, 2, 16>(ctx, a, n_items, item_desc, n_rows, n_adapters, st);
    if (R == 32) return launch_shrink_stream<4, 3, 8>(ctx, a, n_items, item_desc, n_rows, n_adapters, st);
    if (R == 64) return launch_shrink_stream<8, 2, 8>(ctx, a, n_items, item_desc, n_rows, n_adapters, st);
  }
  if (cancelled(ctx)) return MLORA_CANCELLED;
  const int ksplit = shrink_ksplit(ctx, n_items, a.D);
  a.partial = ctx->ws_partial;
  a.counters = ctx->ws_counters;
  if ((int64_t)n_items * ksplit > ctx->ws_partial_items || n_items > ctx->ws_counter_items) return MLORA_ERR_INVALID_ARG;
  LaunchScope scope(ctx, st, KIND_SHRINK);
  switch (R) {
    case 8: launch_shrink_rb<1, 2, 8, 2>(scope.slot < 0, a, n_items, ksplit, st); break;
    case 16: launch_shrink_rb<2, 2, 8, 2>(scope.slot < 0, a, n_items, ksplit, st); break;
    case 32: launch_shrink_rb<4, 2, 8, 2>(scope.slot < 0, a, n_items, ksplit, st); break;
    case 64: launch_shrink_rb<8, 2, 4, 2>(scope.slot < 0, a, n_items, ksplit, st); break;
    case 128:
      if (ctx->drop.thr != 0 && a.item_save) {      // forward with dropout: the mask acts on the rows as they are read
        a.drop = ctx->drop;
        launch_pdl(scope.slot < 0, shrink_kernel<16, 1, 4, 2, true>, dim3(n_items, ksplit, kItemRows / 16), dim3(4 * 32), 0, st, a);
      } else {
        launch_shrink_rb<16, 1, 4, 2>(scope.slot < 0, a, n_items, ksplit, st);
      }
      break;
    default: return MLORA_ERR_UNSUPPORTED;
  }
  return scope.done();
}

// Both gradients of a backward in one launch of the streaming kernel (dB first, then dA).
template <int MB, bool DROP, int CB>
mlora_status_t launch_grad_stream2_d(mlora_ctx* ctx, const mlora_plan* p, const GradArgs& gb, const GradArgs& ga_, int n_slots,
                                     int n_rows, cudaStream_t st) {
  constexpr size_t smem = gw_smem_bytes(CB, MB);
  constexpr int cols = CB * 64;
  static bool attr_set_dev[kMaxDevices] = {};   // per instantiation and device
  bool& attr_set = attr_set_dev[ctx->device];
  auto kern = grad_stream_kernel<MB, DROP, CB>;
  {
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    if (!attr_set) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return MLORA_ERR_CUDA;
      attr_set = true;
    }
  }
  CUtensorMap tQ0, tQ1;
  mlora_status_t ms;
  // (64, rows, D / 64) views: one box = a 64-row tile of a strip as CB swizzled 64-column blocks
  if ((ms = make_tmap_bf16_blocked(ctx, &tQ0, gb.Q, n_rows, gb.D, gb.ldq, GW_ROWS, CB)) != MLORA_OK) return ms;
  if ((ms = make_tmap_bf16_blocked(ctx, &tQ1, ga_.Q, n_rows, ga_.D, ga_.ldq, GW_ROWS, CB)) != MLORA_OK) return ms;
  GradStreamArgs g;
  g.prob[0] = GradProblem{gb.P, gb.scale, gb.G, gb.D, (gb.D + cols - 1) / cols, DropArgs{0, 0, 1.0f}};
  g.prob[1] = GradProblem{ga_.P, ga_.scale, ga_.G, ga_.D, (ga_.D + cols - 1) / cols, ctx->drop};   // dA sees the dropped branch input
  g.n_problems = 2; g.R = gb.R; g.accumulate = gb.accumulate;
  g.slot_adapter = p->slot_adapter; g.slot_blk_off = p->slot_blk_off; g.blk_row0 = p->blk_row0; g.blk_nrows = p->blk_nrows;
  g.n_slots = n_slots; g.status = ctx->status_dev;
  const int groups = n_slots * (g.prob[0].n_strips + g.prob[1].n_strips);
  // One or two fine-tuning adapters leave most SMs without a group: the row blocks of each slot are
  // then dealt out over several CTAs per group (at most one CTA per SM in all, so the partial sums
  // fit the context's workspace), and the last CTA of a group adds the parts in index order.
  int parts = 1;
  if (2 * groups <= ctx->sm_count) {
    int max_blocks = 1;
    for (int sl = 0; sl < n_slots; ++sl) {
      const int nb = p->h.slot_blk_off[sl + 1] - p->h.slot_blk_off[sl];
      max_blocks = nb > max_blocks ? nb : max_blocks;
    }
    parts = ctx->sm_count / groups;
    parts = parts < max_blocks ? parts : max_blocks;
  }
  g.n_parts = parts; g.part_ws = ctx->ws_gpart; g.part_counters = ctx->ws_gcounters;
  const int units = groups * parts;
  const int grid = units < ctx->sm_count ? units : ctx->sm_count;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  LaunchScope scope(ctx, st, KIND_GRAD);
  launch_pdl(scope.slot < 0, kern, dim3(grid), dim3(STREAM_THREADS), smem, st, tQ0, tQ1, g);
  return scope.done();
}

template <int MB, bool DROP>
mlora_status_t launch_grad_stream2_c(mlora_ctx* ctx, const mlora_plan* p, const GradArgs& gb, const GradArgs& ga_, int n_slots,
                                     int n_rows, cudaStream_t st) {
  // 512-column strips unless they leave more than a quarter of the SMs without a group
  const int groups512 = n_slots * ((gb.D + 511) / 512 + (ga_.D + 511) / 512);
  if (4 * groups512 < 3 * ctx->sm_count)
    return launch_grad_stream2_d<MB, DROP, 4>(ctx, p, gb, ga_, n_slots, n_rows, st);
  return launch_grad_stream2_d<MB, DROP, 8>(ctx, p, gb, ga_, n_slots, n_rows, st);
}

template <int MB>
mlora_status_t launch_grad_stream2(mlora_ctx* ctx, const mlora_plan* p, const GradArgs& gb, const GradArgs& ga_, int n_slots,
                                   int n_rows, cudaStream_t st) {
  if constexpr (MB <= 4) {           // dropout is offered up to rank 64 (the streaming kernels' range)
    if (ctx->drop.thr != 0) return launch_grad_stream2_c<MB, true>(ctx, p, gb, ga_, n_slots, n_rows, st);
  }
  return launch_grad_stream2_c<MB, false>(ctx, p, gb, ga_, n_slots, n_rows, st);
}

// U = X A^T (forward, with the activation save) or V = s dY B^T (backward) on the tcgen05 kernels: the rows come
// as blocks of <= 128 consecutive rows of one adapter.  `fa` carries what the finish kernel writes.
template <int R>
mlora_status_t launch_shrink_tc(mlora_ctx* ctx, const RowSpace& hs, const DevRowSpace& ds, const void* In, int64_t ld_in,
                                int n_rows, int D, const void* P_all, int n_adapters, stc::FinArgs fa, cudaStream_t st) {
  using C = stc::Cfg<R>;
  static bool attr_set_dev[kMaxDevices] = {};   // per instantiation and device
  bool& attr_set = attr_set_dev[ctx->device];
  auto kern = stc::shrink_tc_kernel<R>;
  {
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    if (!attr_set) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES) != cudaSuccess) return MLORA_ERR_CUDA;
      attr_set = true;
    }
  }
  CUtensorMap tQ, tB, tB16, tB32, tB64;
  mlora_status_t ms;
  if ((ms = make_tmap_bf16_blocked(ctx, &tQ, In, n_rows, D, ld_in, stc::ROWS, C::CB)) != MLORA_OK) return ms;
  if ((ms = make_tmap_bf16_blocked(ctx, &tB, P_all, (uint64_t)n_adapters * R, D, D, C::RP, C::CB)) != MLORA_OK) return ms;
  tB16 = tB; tB32 = tB; tB64 = tB;
  if (ds.tcb_width) {      // plans with per-adapter ranks: a block reads only as many rows of its adapter's matrix as the rank needs
    if ((ms = make_tmap_bf16_blocked(ctx, &tB16, P_all, (uint64_t)n_adapters * R, D, D, 16, C::CB)) != MLORA_OK) return ms;
    if (C::RP > 32 && (ms = make_tmap_bf16_blocked(ctx, &tB32, P_all, (uint64_t)n_adapters * R, D, D, 32, C::CB)) != MLORA_OK) return ms;
    if (C::RP > 64 && (ms = make_tmap_bf16_blocked(ctx, &tB64, P_all, (uint64_t)n_adapters * R, D, D, 64, C::CB)) != MLORA_OK) return ms;
  }
  stc::Args a;
  a.blk_row0 = ds.tcb_row0; a.blk_nrows = ds.tcb_nrows; a.blk_adapter = ds.tcb_adapter; a.blk_width = ds.tcb_width;
  a.NB = (int)hs.tcb_row0.size(); a.NS = (D + C::COLS - 1) / C::COLS;
  a.part_ws = ctx->ws_tc_part; a.status = ctx->status_dev;
  const int64_t tiles = (int64_t)a.NB * a.NS;
  const int grid = tiles < ctx->sm_count ? (int)tiles : ctx->sm_count;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  {
    LaunchScope scope(ctx, st, KIND_SHRINK);
    launch_pdl(scope.slot < 0, kern, dim3(grid), dim3(stc::THREADS), C::SMEM_BYTES, st, tQ, tB, tB16, tB32, tB64, a);
    if ((ms = scope.done()) != MLORA_OK) return ms;
  }
  fa.blk_row0 = a.blk_row0; fa.blk_nrows = a.blk_nrows; fa.blk_adapter = a.blk_adapter; fa.blk_width = a.blk_width;
  fa.NB = a.NB; fa.NS = a.NS; fa.G = grid; fa.part_ws = ctx->ws_tc_part;
  const int zero_ctas = fa.pbd.pbd ? (fa.pbd.n_zero_rows + C::FIN_ROWS - 1) / C::FIN_ROWS : 0;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  LaunchScope scope(ctx, st, KIND_SHRINK);
  launch_pdl(scope.slot < 0, stc::shrink_tc_finish_kernel<R>, dim3(a.NB + zero_ctas, stc::ROWS / C::FIN_ROWS), dim3(C::FIN_THREADS), 0,
             st, fa);
  return scope.done();
}

// Can this row space run on the tensor-core shrink?  Blocks that are nearly empty waste the 128-row MMA: below four
// rows per block on average at rank 128 (where the alternative is the per-item kernel: 256 adapters on 2048 rows,
// 11 rows per block, 45 + 15 us against 85), eight at the lower ranks (where it is the streaming kernel that gathers
// rows by adapter: 512 single-row blocks beside 2048 fine-tuning rows at rank 32, 83 + 23 us against 41), the
// mma.sync kernels are the better choice.
inline bool shrink_tc_fits(const mlora_ctx* ctx, const RowSpace& hs, int n_rows, int D, int rank) {
  const int64_t NB = (int64_t)hs.tcb_row0.size();
  if (NB < 1 || D % 64 != 0 || n_rows > ctx->ws_rows || !ctx->ws_tc_part) return false;
  if ((rank >= 128 ? 4 : 8) * NB > (int64_t)hs.item_rows.size()) return false;
  return NB * ((D + 127) / 128) < (1 << 30) && NB + (int64_t)hs.zero_rows2.size() / 8 + 1 < (1 << 30);
}

inline mlora_status_t launch_shrink_tc_any(mlora_ctx* ctx, int rank, const RowSpace& hs, const DevRowSpace& ds, const void* In,
                                           int64_t ld_in, int n_rows, int D, const void* P_all, int n_adapters,
                                           const stc::FinArgs& fa, cudaStream_t st) {
  switch (rank) {
    case 8: return launch_shrink_tc<8>(ctx, hs, ds, In, ld_in, n_rows, D, P_all, n_adapters, fa, st);
    case 16: return launch_shrink_tc<16>(ctx, hs, ds, In, ld_in, n_rows, D, P_all, n_adapters, fa, st);
    case 32: return launch_shrink_tc<32>(ctx, hs, ds, In, ld_in, n_rows, D, P_all, n_adapters, fa, st);
    case 64: return launch_shrink_tc<64>(ctx, hs, ds, In, ld_in, n_rows, D, P_all, n_adapters, fa, st);
    case 128: return launch_shrink_tc<128>(ctx, hs, ds, In, ld_in, n_rows, D, P_all, n_adapters, fa, st);
    default: return MLORA_ERR_UNSUPPORTED;
  }
}

// Both gradients on the tcgen05 kernel: can this call use it?  (A slot without rows gets its zeros from the
// other kernels; the counters have a fixed size.)
template <int R>
bool grad_tc_fits(const mlora_layer_t* L, const mlora_plan* p) {
  using C = gtc::Cfg<R>;
  const HostPlan& h = p->h;
  const int n_slots = (int)h.ft_adapters.size();
  if (n_slots < 1) return false;
  for (int sl = 0; sl < n_slots; ++sl)
    if (h.slot_blk_off[sl + 1] == h.slot_blk_off[sl]) return false;
  const int64_t NB = (int64_t)h.blk_row0.size();
  const int64_t NS0 = (L->d_out + C::COLS - 1) / C::COLS, NS1 = (L->d_in + C::COLS - 1) / C::COLS;
  if (1 + n_slots * (NS0 + NS1) > kTcCounters) return false;
  return NB * (NS0 + NS1) < (1 << 30);
}

// First tile of CTA c's range in the combined list, with the ends moved down to strip boundaries (what the
// kernel does when `snap` is set): used to decide whether snapping keeps the ranges even.
int64_t grad_tc_snapped_begin(const HostPlan& h, int64_t NS0, int64_t NS1, int c, int G) {
  const int64_t NB = (int64_t)h.blk_row0.size(), N0 = NB * NS0, N = NB * (NS0 + NS1);
  int64_t g = (int64_t)c * N / G;
  if (g >= N) return N;
  const int64_t NS = g >= N0 ? NS1 : NS0, t = g >= N0 ? g - N0 : g;
  size_t slot = 0;
  while ((int64_t)h.slot_blk_off[slot + 1] * NS <= t) ++slot;
  const int64_t nb = h.slot_blk_off[slot + 1] - h.slot_blk_off[slot];
  return g - (t - (int64_t)h.slot_blk_off[slot] * NS) % nb;
}

template <int R>
mlora_status_t launch_grad_tc(mlora_ctx* ctx, const mlora_layer_t* L, const mlora_plan* p, const void* dY, int64_t lddy,
                              const void* x_save, const float* u_save, float* dA, float* dB, int accumulate, cudaStream_t st) {
  using C = gtc::Cfg<R>;
  const HostPlan& h = p->h;
  static bool attr_set_dev[kMaxDevices] = {};   // per instantiation and device
  bool& attr_set = attr_set_dev[ctx->device];
  auto kern = gtc::grad_tc_kernel<R>;
  {
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    if (!attr_set) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES) != cudaSuccess) return MLORA_ERR_CUDA;
      attr_set = true;
    }
  }
  CUtensorMap tQ0, tQ1;
  mlora_status_t ms;
  // (64, rows, D / 64) views: one box = a 128-row tile as CB swizzled 64-column blocks
  if ((ms = make_tmap_bf16_blocked(ctx, &tQ0, dY, h.ft_rows, L->d_out, lddy, gtc::ROWS, C::CB)) != MLORA_OK) return ms;
  if ((ms = make_tmap_bf16_blocked(ctx, &tQ1, x_save, h.ft_rows, L->d_in, L->d_in, gtc::ROWS, C::CB)) != MLORA_OK) return ms;
  gtc::Args a;
  const int NS0 = (L->d_out + C::COLS - 1) / C::COLS, NS1 = (L->d_in + C::COLS - 1) / C::COLS;
  a.prob[0] = gtc::Problem{u_save, L->scale, dB, L->d_out, NS0};       // dB = (s u)^T dY
  a.prob[1] = gtc::Problem{ctx->ws_p, nullptr, dA, L->d_in, NS1};      // dA = V^T x, V already carries s
  a.slot_adapter = p->slot_adapter; a.slot_blk_off = p->slot_blk_off; a.blk_row0 = p->blk_row0; a.blk_nrows = p->blk_nrows;
  a.n_slots = (int)h.ft_adapters.size(); a.NB = (int)h.blk_row0.size();
  a.part_ws = ctx->ws_gpart; a.counters = ctx->ws_tc_counters; a.n_counters = 1 + a.n_slots * (NS0 + NS1);
  a.accumulate = accumulate; a.status = ctx->status_dev;
  const int64_t tiles = (int64_t)a.NB * (NS0 + NS1);
  const int grid = tiles < ctx->sm_count ? (int)tiles : ctx->sm_count;
  // Ranges that end at strip boundaries need no partial sums; taken when they stay nearly as even as plain ranges.
  int64_t most_plain = 0, most_snapped = 0;
  for (int c = 0; c < grid; ++c) {
    const int64_t plain = (int64_t)(c + 1) * tiles / grid - (int64_t)c * tiles / grid;
    const int64_t snapped = grad_tc_snapped_begin(h, NS0, NS1, c + 1, grid) - grad_tc_snapped_begin(h, NS0, NS1, c, grid);
    most_plain = plain > most_plain ? plain : most_plain;
    most_snapped = snapped > most_snapped ? snapped : most_snapped;
  }
  a.snap = (8 * most_snapped <= 9 * most_plain) ? 1 : 0;
  a.pop = nullptr;
  a.slot_width = nullptr;
  if (a.NB <= ctx->ws_pop_blocks && ctx->ws_pop) {     // both problems' operands once per block, ahead of the kernel
    a.slot_width = p->slot_width;                      // (ranked plans: only the rows of a gradient that exist)
    if (cancelled(ctx)) return MLORA_CANCELLED;
    LaunchScope scope(ctx, st, KIND_GRAD);
    launch_pdl(scope.slot < 0, gtc::psplit_kernel<R>, dim3(a.NB, 2, R / gtc::psplit_cols(R)), dim3(128), 0, st, a, ctx->ws_pop);
    if ((ms = scope.done()) != MLORA_OK) return ms;
    a.pop = ctx->ws_pop;
  }
  if (cancelled(ctx)) return MLORA_CANCELLED;
  LaunchScope scope(ctx, st, KIND_GRAD);
  launch_pdl(scope.slot < 0, kern, dim3(grid), dim3(gtc::THREADS), C::SMEM_BYTES, st, tQ0, tQ1, a);
  return scope.done();
}

mlora_status_t launch_grad(mlora_ctx* ctx, const mlora_plan* p, const GradArgs& a, int n_slots, int n_rows,
                           cudaStream_t st) {
  if (n_slots <= 0) return MLORA_OK;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  constexpr int smem1 = (GRAD_THREADS / 32) * 16 * 65 * 4, smem2 = 2 * smem1;
  static bool attr_set_dev[kMaxDevices] = {};   // per instantiation and device
  bool& attr_set = attr_set_dev[ctx->device];
  {
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    if (!attr_set) {
      if (cudaFuncSetAttribute(grad_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2) != cudaSuccess ||
          cudaFuncSetAttribute(grad_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2) != cudaSuccess)
        return MLORA_ERR_CUDA;
      attr_set = true;
    }
  }
  LaunchScope scope(ctx, st, KIND_GRAD);
  if (a.R <= 16) {
    launch_pdl(scope.slot < 0, grad_kernel<1>, dim3(a.D / 64, n_slots, 1), dim3(GRAD_THREADS), smem1, st, a);
  } else {
    if (a.drop.thr != 0)
      launch_pdl(scope.slot < 0, grad_kernel<2, true>, dim3(a.D / 64, n_slots, (a.R + 31) / 32), dim3(GRAD_THREADS), smem2, st, a);
    else
      launch_pdl(scope.slot < 0, grad_kernel<2>, dim3(a.D / 64, n_slots, (a.R + 31) / 32), dim3(GRAD_THREADS), smem2, st, a);
  }
  return scope.done();
}

// dX += keep * (V A_a) / (1 - p): the low-rank part of the input gradient under dropout, after the
// base product has been written by the GEMM.
mlora_status_t launch_expand_mask(mlora_ctx* ctx, const mlora_layer_t* L, const DevRowSpace& ds, void* dX, int64_t lddx,
                                  int n_rows, cudaStream_t st) {
  if (n_rows <= 0) return MLORA_OK;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  ExpandMaskArgs a;
  a.V = ctx->ws_p; a.R = L->rank; a.A_all = (const __nv_bfloat16*)L->A_all; a.row_adapter = ds.row_adapter;
  a.dX = (__nv_bfloat16*)dX; a.lddx = lddx; a.D = L->d_in; a.n_rows = n_rows; a.drop = ctx->drop;
  LaunchScope scope(ctx, st, KIND_SHRINK);
  launch_pdl(scope.slot < 0, expand_mask_kernel, dim3((n_rows + EM_ROWS - 1) / EM_ROWS, (L->d_in / 8 + 127) / 128), dim3(128), 0, st, a);
  return scope.done();
}

template <int R, bool W_KMAJOR>
mlora_status_t launch_gemm_r(mlora_ctx* ctx, const CUtensorMap& tIn, const CUtensorMap& tW, const CUtensorMap& tL,
                             const CUtensorMap& tOut, const GemmArgs& g, cudaStream_t st) {
  static bool attr_set_dev[kMaxDevices] = {};   // per instantiation and device: the attribute belongs to the device's context
  bool& attr_set = attr_set_dev[ctx->device];
  auto kern = gemm_lora_kernel<R, W_KMAJOR>;
  {
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    if (!attr_set) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM_BYTES) != cudaSuccess)
        return MLORA_ERR_CUDA;
      attr_set = true;
    }
  }
  if (cancelled(ctx)) return MLORA_CANCELLED;
  const int grid = g.n_units < ctx->sm_count ? g.n_units : ctx->sm_count;
  LaunchScope scope(ctx, st, W_KMAJOR ? KIND_GEMM_BWD : KIND_GEMM_FWD);
  launch_pdl(scope.slot < 0, kern, dim3(grid), dim3(GEMM_THREADS), GEMM_SMEM_BYTES, st, tIn, tW, tL, tOut, g);
  return scope.done();
}

// Two-SM kernel: grid = 2 x (number of CTA pairs that can be resident at once).
template <int R, bool W_KMAJOR>
mlora_status_t launch_gemm2_r(mlora_ctx* ctx, const CUtensorMap& tIn, const CUtensorMap& tW, const CUtensorMap& tL,
                              const CUtensorMap& tOut, const CUtensorMap& tPbd, const GemmArgs& g, cudaStream_t st) {
  static int max_pairs_dev[kMaxDevices] = {};   // per instantiation and device
  int& max_pairs = max_pairs_dev[ctx->device];
  auto kern = gemm2_lora_kernel<R, W_KMAJOR>;
  std::unique_lock<std::mutex> attr_lock(g_attr_mutex);
  if (max_pairs == 0) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM2_SMEM_BYTES) != cudaSuccess)
      return MLORA_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ctx->sm_count); cfg.blockDim = dim3(GEMM2_THREADS); cfg.dynamicSmemBytes = GEMM2_SMEM_BYTES;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) { cudaGetLastError(); return MLORA_ERR_CUDA; }
    max_pairs = n;
  }
  const int pairs = g.n_units < max_pairs ? g.n_units : max_pairs;
  attr_lock.unlock();
  if (cancelled(ctx)) return MLORA_CANCELLED;
  GemmArgs ga = g;
  if (ga.unit_list && ga.sched_pairs != pairs) ga.unit_list = nullptr;   // the list was made for another grid
  LaunchScope scope(ctx, st, W_KMAJOR ? KIND_GEMM_BWD : KIND_GEMM_FWD);
  launch_pdl_pairs(scope.slot < 0, kern, dim3(2 * pairs), dim3(GEMM2_THREADS), GEMM2_SMEM_BYTES, st, tIn, tW, tL, tOut, tPbd, ga);
  return scope.done();
}

template <bool W_KMAJOR>
mlora_status_t launch_gemm2(mlora_ctx* ctx, int R, const CUtensorMap& tIn, const CUtensorMap& tW, const CUtensorMap& tL,
                            const CUtensorMap& tOut, const CUtensorMap& tPbd, const GemmArgs& g, cudaStream_t st) {
  switch (R) {
    case 8: return launch_gemm2_r<8, W_KMAJOR>(ctx, tIn, tW, tL, tOut, tPbd, g, st);
    case 16: return launch_gemm2_r<16, W_KMAJOR>(ctx, tIn, tW, tL, tOut, tPbd, g, st);
    case 32: return launch_gemm2_r<32, W_KMAJOR>(ctx, tIn, tW, tL, tOut, tPbd, g, st);
    case 64: return launch_gemm2_r<64, W_KMAJOR>(ctx, tIn, tW, tL, tOut, tPbd, g, st);
    case 128: return launch_gemm2_r<128, W_KMAJOR>(ctx, tIn, tW, tL, tOut, tPbd, g, st);
    default: return MLORA_ERR_UNSUPPORTED;
  }
}

template <bool W_KMAJOR>
mlora_status_t launch_gemm(mlora_ctx* ctx, int R, const CUtensorMap& tIn, const CUtensorMap& tW, const CUtensorMap& tL,
                           const CUtensorMap& tOut, const GemmArgs& g, cudaStream_t st) {
  switch (R) {
    case 8: return launch_gemm_r<8, W_KMAJOR>(ctx, tIn, tW, tL, tOut, g, st);
    case 16: return launch_gemm_r<16, W_KMAJOR>(ctx, tIn, tW, tL, tOut, g, st);
    case 32: return launch_gemm_r<32, W_KMAJOR>(ctx, tIn, tW, tL, tOut, g, st);
    case 64: return launch_gemm_r<64, W_KMAJOR>(ctx, tIn, tW, tL, tOut, g, st);
    case 128: return launch_gemm_r<128, W_KMAJOR>(ctx, tIn, tW, tL, tOut, g, st);
    default: return MLORA_ERR_UNSUPPORTED;
  }
}

// Units of the two-SM GEMM dealt out by cost.  The kernel's default - pair p takes units p, p + pairs, ... -
// assumes tiles of equal cost; a 256-row tile with G adapter groups carries ceil(G r / 64) low-rank
// K-blocks on top of its K / 64 main ones, so a batch with one tile of 135 single-row adapters next to
// tiles of one group (rank 128: 334 against 66 blocks) leaves the pairs that meet the heavy tiles with
// 1.5 times the mean load.  Here the units go, heaviest first, to the pair with the least load so far
// (each pair's units then in tile order).  The list is made once per plan and shape on the host and
// copied behind the plan's tables; g.unit_list stays null when round robin is within 3% of it, when the
// plan reserved no room (even row spaces), or when the stream is being captured before the list exists.
void balanced_units(mlora_ctx* ctx, const RowSpace& hs, const DevRowSpace& ds, int R, int kblocks, GemmArgs& g,
                    cudaStream_t st) {
  g.unit_list = nullptr; g.sched_pairs = 0;
  SchedCache* sc = ds.sched;
  if (!sc || !sc->dev || !sc->mirror || ctx->no_unit_lists || !g.lora_enabled) return;
  if ((int64_t)sc->lc_spread * R < 2 * 64) return;          // tiles differ by less than two K-blocks
  const int pairs = g.n_units < ctx->sm_count / 2 ? g.n_units : ctx->sm_count / 2;
  if (pairs < 2 || g.n_units + pairs + 1 > kSchedCap) return;
  std::lock_guard<std::mutex> lock(sc->mu);
  SchedEntry* e = nullptr;
  int slot = 0;
  for (; slot < sc->n; ++slot) {
    SchedEntry& x = sc->e[slot];
    if (x.n_ntiles == g.n_ntiles && x.kblocks == kblocks && x.rank == R && x.pairs == pairs && x.n_whole == g.n_whole &&
        x.n_tail == g.n_tail && x.split_k == g.split_k && x.group_m == g.group_m) { e = &x; break; }
  }
  if (!e) {
    if (sc->n >= kSchedSlots) return;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) { cudaGetLastError(); return; }
    // cost of every unit in K-blocks (+2: accumulator hand-over and the first loads of a tile)
    std::vector<int32_t> cost(g.n_units);
    for (int u = 0; u < g.n_units; ++u) {
      int tile, ks, sk, mt, nt;
      gemm2_unit(g, u, tile, ks, sk);
      gemm2_tile(g, tile, mt, nt);
      const int G = hs.tile2_grp_off[mt + 1] - hs.tile2_grp_off[mt];
      const int LC = ((g.piece_src ? hs.tile2_cols[mt] : G * R) + 63) / 64;
      const int kb = (int)((int64_t)(ks + 1) * kblocks / sk) - (int)((int64_t)ks * kblocks / sk);
      const int lc = (int)((int64_t)(ks + 1) * LC / sk) - (int)((int64_t)ks * LC / sk);
      cost[u] = kb + lc + 2;
    }
    std::vector<int64_t> rr(pairs, 0);
    for (int u = 0; u < g.n_units; ++u) rr[u % pairs] += cost[u];
    const int64_t rr_max = *std::max_element(rr.begin(), rr.end());
    std::vector<int32_t> order(g.n_units);
    for (int u = 0; u < g.n_units; ++u) order[u] = u;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost[a] > cost[b]; });
    typedef std::pair<int64_t, int> Load;                     // (load, pair): the least loaded pair, lowest index first
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int p = 0; p < pairs; ++p) heap.push(Load(0, p));
    std::vector<std::vector<int32_t>> mine(pairs);
    int64_t lpt_max = 0;
    for (int u : order) {
      Load l = heap.top(); heap.pop();
      l.first += cost[u];
      mine[l.second].push_back(u);
      lpt_max = l.first > lpt_max ? l.first : lpt_max;
      heap.push(l);
    }
    e = &sc->e[sc->n];
    e->n_ntiles = g.n_ntiles; e->kblocks = kblocks; e->rank = R; e->pairs = pairs; e->n_whole = g.n_whole;
    e->n_tail = g.n_tail; e->split_k = g.split_k; e->group_m = g.group_m;
    e->use = 100 * lpt_max < 97 * rr_max;
    if (std::getenv("MLORA_DEBUG"))
      std::fprintf(stderr, "mlora: unit list for %d x %d tiles, %d K-blocks, rank %d: round robin %lld, by cost %lld blocks -> %s\n",
                   g.n_mtiles, g.n_ntiles, kblocks, R, (long long)rr_max, (long long)lpt_max, e->use ? "list" : "round robin");
    slot = sc->n;
    if (e->use) {
      int32_t* list = sc->mirror + (size_t)slot * kSchedCap;      // offsets (into this same array), then each pair's units in tile order
      int32_t at = pairs + 1;
      for (int p = 0; p < pairs; ++p) {
        std::sort(mine[p].begin(), mine[p].end());
        list[p] = at;
        for (int32_t u : mine[p]) list[at++] = u;
      }
      list[pairs] = at;
      if (cudaEventCreateWithFlags(&e->filled, cudaEventDisableTiming) != cudaSuccess ||
          cudaMemcpyAsync(sc->dev + (size_t)slot * kSchedCap, list, (size_t)at * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess ||
          cudaEventRecord(e->filled, st) != cudaSuccess) {
        cudaGetLastError();
        e->use = false;
      }
      e->stream = st;
    }
    sc->n++;
  }
  if (!e->use) return;
  if (e->stream != st && e->filled) {        // another stream than the one that filled the list: order behind the copy
    if (cudaEventQuery(e->filled) != cudaSuccess) {
      cudaGetLastError();
      if (cudaStreamWaitEvent(st, e->filled, 0) != cudaSuccess) { cudaGetLastError(); return; }
    }
  }
  g.unit_list = sc->dev + (size_t)slot * kSchedCap;
  g.sched_pairs = e->pairs;
}

// A plan made with per-adapter ranks serves layers whose padded rank is a multiple of 16 and at least every adapter's own.
inline bool ranked_plan_fits(const HostPlan& h, const mlora_layer_t* L) {
  if (h.adapter_rank.empty()) return true;
  if (L->rank % 16 != 0) return false;
  for (int32_t r : h.adapter_rank)
    if (r > L->rank) return false;
  return true;
}
inline void set_ranked(PbdArgs& pa, const DevRowSpace& ds) {
  pa.grp2_col = ds.grp2_col; pa.grp2_width = ds.grp2_width; pa.tile2_cols = ds.tile2_cols;
}

// Out = In Wop + (scale) P L over one row space, tensor-core path.
template <bool W_KMAJOR>
mlora_status_t gemm_bf16(mlora_ctx* ctx, const mlora_layer_t* L, const RowSpace& hs, const DevRowSpace& ds,
                         const void* In, int64_t ld_in, void* Out, int64_t ld_out, const void* L_all,
                         const float* P, const float* scale, int M, int N, int K, cudaStream_t st, bool lora = true) {
  CUtensorMap tIn, tW, tL, tOut;
  mlora_status_t s;
  if ((s = make_tmap_bf16(ctx, &tIn, In, K, M, ld_in, GEMM_BK, GEMM_BM)) != MLORA_OK) return s;
  if (W_KMAJOR) {   // W [N rows, K cols] (the stored [d_in, d_out] matrix read as the transposed operand)
    if ((s = make_tmap_bf16(ctx, &tW, L->W, K, N, L->ldw, GEMM_BK, GEMM_BN / 2)) != MLORA_OK) return s;
  } else {          // W [K rows, N cols]
    if ((s = make_tmap_bf16_blocked(ctx, &tW, L->W, K, N, L->ldw, GEMM_BK, 2)) != MLORA_OK) return s;
  }
  const int R = L->rank;
  const bool ranked = ds.piece_src != nullptr && ctx->gemm_pairs;    // B-side rows of the low-rank blocks come as 16-row pieces
  if ((s = make_tmap_bf16_blocked(ctx, &tL, L_all, (uint64_t)L->n_adapters * R, N, N, ranked ? 16 : (R < 64 ? R : 64), 1)) != MLORA_OK)
    return s;
  if ((s = make_tmap_bf16(ctx, &tOut, Out, N, M, ld_out, 64, 32)) != MLORA_OK) return s;
  GemmArgs g;
  g.M = M; g.N = N; g.K = K; g.split_k = 1; g.ws_splitk = nullptr; g.unit_list = nullptr; g.sched_pairs = 0;
  g.tile_cols = ranked ? ds.tile2_cols : nullptr; g.tile_piece_off = ranked ? ds.tile2_piece_off : nullptr;
  g.piece_src = ranked ? ds.piece_src : nullptr;
  // Long contractions with many row tiles: the operand panels of one wave of tiles no longer fit the
  // L2 together with their neighbours', so the tiles are walked in bands of 8 row tiles (a wave then
  // covers about 8 x 9 tiles and streams 17 panels instead of 16 + 5 per 74 tiles; measured +2% on
  // 4096 x 14336 -> 4096 under sustained load, -2% on short contractions, hence the condition).
  g.group_m = (K >= 8192 && (M + GEMM2_BM - 1) / GEMM2_BM >= 16) ? 8 : 0;
  if (ctx->gemm_pairs) {            // two-SM kernel: 256-row tiles and their group tables
    g.n_mtiles = (M + GEMM2_BM - 1) / GEMM2_BM;
    g.n_ntiles = (N + GEMM2_BN - 1) / GEMM2_BN;
    // Few tiles for the CTA pairs there are (small batches, the backward of one 256-token fine-tuning
    // batch): cut K into slices of at least 16 K-blocks that run on different pairs; the fp32 partials
    // are summed by a small kernel afterwards (≈8 µs with its launch, hence the bound on what the split
    // has to save).
    const int tiles = g.n_mtiles * g.n_ntiles, pairs = ctx->sm_count / 2, kblocks = (K + GEMM_BK - 1) / GEMM_BK;
    const size_t tile_ws = (size_t)GEMM2_BM * GEMM2_BN * sizeof(float);
    int sk = 1, n_tail = 0;
    if (2 * tiles <= pairs && kblocks >= 64 && !ctx->no_split_k) {          // every tile is split
      sk = pairs / tiles;
      sk = sk < kblocks / 16 ? sk : kblocks / 16;
      sk = sk < 8 ? sk : 8;
      n_tail = tiles;
      // the same bound as for the last wave below (4096 -> 4096 backward of 256 rows, 16 tiles in
      // four slices: 42.6 -> 36.3 µs for the whole call; two slices of such a product do not pay)
      if (sk < 2 || (int64_t)kblocks * (sk - 1) < 40 * (int64_t)sk) { sk = 1; n_tail = 0; }
    } else if (tiles > pairs && !ctx->no_split_k) {
      // More tiles than CTA pairs, and the last wave fills at most half of them: only its tiles are
      // cut along K (slices of at least 16 K-blocks), so that the wave takes 1 / slices of a tile's
      // time.  E.g. 160 tiles on 74 pairs: 12 tail tiles in 6 slices, 2.17 instead of 3 tile times.
      const int rem = tiles % pairs;
      if (rem > 0 && 2 * rem <= pairs && kblocks >= 32) {
        sk = pairs / rem;
        sk = sk < kblocks / 16 ? sk : kblocks / 16;
        sk = sk < 8 ? sk : 8;
        n_tail = rem;
        // Worth it only if the K-blocks the last wave no longer waits for (≈0.4 µs each) outweigh the
        // reduction kernel and the fp32 partial traffic (≈8 µs): the bound below keeps out e.g. a
        // 4096-deep product with a half-full last wave (two slices: 103 -> 101 + 8.6 µs) and lets in
        // a 4096-deep one with 8 tail tiles in four slices (330 -> 314 + 7.7 µs) and the 14336-deep
        // ones (343 -> 305 + 8.6 µs; 13824-deep with 12 tail tiles 255 -> 177 + 8.7 µs).
        if (sk < 2 || (int64_t)kblocks * (sk - 1) < 40 * (int64_t)sk) { sk = 1; n_tail = 0; }
      }
    }
    while (sk > 1 && (size_t)sk * n_tail * tile_ws > kSplitKBytes) --sk;
    if (sk <= 1) { sk = 1; n_tail = 0; }
    g.split_k = sk; g.n_tail = n_tail; g.n_whole = tiles - n_tail; g.ws_splitk = ctx->ws_splitk;
    g.n_full = g.n_units = g.n_whole + n_tail * sk;
    g.lora_enabled = (lora && !hs.grp2_adapter.empty()) ? 1 : 0;
    g.row_grp = ds.row_grp2; g.row_adapter = ds.row_adapter;
    g.tile_grp_off = ds.tile2_grp_off; g.grp_adapter = ds.grp2_adapter;
    g.P = P; g.scale = scale; g.status = ctx->status_dev;
    balanced_units(ctx, hs, ds, R, kblocks, g, st);
    CUtensorMap tPbd;
    const uint64_t slots = g.lora_enabled ? 2 * (uint64_t)hs.grp2_adapter.size() : 1;
    if ((s = make_tmap_bf16(ctx, &tPbd, ctx->ws_pbd ? (const void*)ctx->ws_pbd : In, 64, slots * 256, 64, 64, 128)) != MLORA_OK)
      return s;
    if ((s = launch_gemm2<W_KMAJOR>(ctx, R, tIn, tW, tL, tOut, tPbd, g, st)) != MLORA_OK || sk == 1) return s;
    if (cancelled(ctx)) return MLORA_CANCELLED;
    LaunchScope scope(ctx, st, KIND_REDUCE);
    launch_pdl(scope.slot < 0, splitk_reduce_kernel, dim3((unsigned)(n_tail * 32)), dim3(256), 0, st, g,
               (__nv_bfloat16*)Out, ld_out);
    return scope.done();
  }
  g.n_mtiles = (M + GEMM_BM - 1) / GEMM_BM;
  g.n_ntiles = (N + GEMM_BN - 1) / GEMM_BN;
  // The last wave of tiles usually fills only part of the SMs; when it fills at most half, its
  // tiles are cut into two 128 x 128 halves so that it takes half as long.
  {
    const int tiles = g.n_mtiles * g.n_ntiles;
    const int sms = ctx->sm_count;
    const int rem = tiles % sms;
    const bool split = tiles > sms && rem > 0 && 2 * rem <= sms;
    g.n_full = split ? tiles - rem : tiles;
    g.n_units = split ? tiles + rem : tiles;
  }
  g.lora_enabled = (lora && !hs.grp_adapter.empty()) ? 1 : 0;
  g.row_grp = ds.row_grp; g.row_adapter = ds.row_adapter;
  g.tile_grp_off = ds.tile_grp_off; g.grp_adapter = ds.grp_adapter;
  g.P = P; g.scale = scale; g.status = ctx->status_dev;
  return launch_gemm<W_KMAJOR>(ctx, R, tIn, tW, tL, tOut, g, st);
}

// ---- generic (fp32 / cross-check) launches --------------------------------------------------
template <typename T>
mlora_status_t simt_shrink(mlora_ctx* ctx, const T* In, int64_t ld_in, int D, int R, const T* P_all,
                           const float* scale, const DevRowSpace& ds, float* Out, T* x_save, float* u_save,
                           int64_t save_base, int n_rows, int n_adapters, const DropArgs& drop, cudaStream_t st) {
  if (n_rows <= 0) return MLORA_OK;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  const int64_t warps = (int64_t)n_rows * R;
  const int blocks = (int)((warps * 32 + 255) / 256);
  LaunchScope scope(ctx, st, KIND_SIMT);
  simt::shrink_kernel<T><<<blocks, 256, 0, st>>>(In, ld_in, D, R, P_all, scale, ds.row_adapter, ds.row_save, Out,
                                                 x_save, u_save, save_base, n_rows, n_adapters, drop);
  return scope.done();
}

template <typename T, bool W_KMAJOR>
mlora_status_t simt_gemm(mlora_ctx* ctx, const T* In, int64_t ld_in, const T* W, int64_t ldw, const T* L_all,
                         const float* P, const float* scale, const DevRowSpace& ds, T* Out, int64_t ld_out, int M,
                         int N, int K, int R, int n_adapters, const DropArgs& drop, cudaStream_t st) {
  if (M <= 0) return MLORA_OK;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  dim3 grid((N + 31) / 32, (M + 31) / 32), block(32, 32);
  LaunchScope scope(ctx, st, KIND_SIMT);
  simt::gemm_lora_kernel<T, W_KMAJOR><<<grid, block, 0, st>>>(In, ld_in, W, ldw, L_all, P, scale, ds.row_adapter, Out,
                                                              ld_out, M, N, K, R, n_adapters, drop);
  return scope.done();
}

template <typename T>
mlora_status_t simt_grad(mlora_ctx* ctx, const mlora_plan* p, const float* P, int R, const float* scale, const T* Q,
                         int64_t ldq, int D, float* G, int accumulate, const DropArgs& drop, cudaStream_t st) {
  const int n_slots = (int)p->h.ft_adapters.size();
  if (n_slots <= 0) return MLORA_OK;
  if (cancelled(ctx)) return MLORA_CANCELLED;
  dim3 grid((D + 127) / 128, R, n_slots);
  LaunchScope scope(ctx, st, KIND_SIMT);
  simt::grad_kernel<T><<<grid, 128, 0, st>>>(P, R, scale, Q, ldq, D, G, p->slot_chunk_off, p->chunk_row0,
                                             p->chunk_nrows, p->slot_adapter, accumulate, drop);
  return scope.done();
}

template <typename T>
mlora_status_t forward_simt(mlora_ctx* ctx, const mlora_layer_t* L, const mlora_plan* p, const void* X, int64_t ldx,
                            void* Y, int64_t ldy, void* x_save, float* u_save, int64_t save_base, cudaStream_t st) {
  const DropArgs off = {0, 0, 1.0f};
  mlora_status_t s = simt_shrink<T>(ctx, (const T*)X, ldx, L->d_in, L->rank, (const T*)L->A_all, nullptr, p->fwd,
                                    ctx->ws_p, (T*)x_save, u_save, save_base, p->h.n_rows, L->n_adapters, ctx->drop, st);
  if (s != MLORA_OK) return s;
  return simt_gemm<T, false>(ctx, (const T*)X, ldx, (const T*)L->W, L->ldw, (const T*)L->B_all, ctx->ws_p, L->scale,
                             p->fwd, (T*)Y, ldy, p->h.n_rows, L->d_out, L->d_in, L->rank, L->n_adapters, off, st);
}

template <typename T>
mlora_status_t backward_simt(mlora_ctx* ctx, const mlora_layer_t* L, const mlora_plan* p, const void* dY, int64_t lddy,
                             const void* x_save, const float* u_save, float* dA, float* dB, void* dX, int64_t lddx,
                             int accumulate, cudaStream_t st) {
  const int Tft = p->h.ft_rows;
  const DropArgs off = {0, 0, 1.0f};
  mlora_status_t s = simt_shrink<T>(ctx, (const T*)dY, lddy, L->d_out, L->rank, (const T*)L->B_all, L->scale, p->bwd,
                                    ctx->ws_p, (T*)nullptr, nullptr, 0, Tft, L->n_adapters, off, st);
  if (s != MLORA_OK) return s;
  if ((s = simt_grad<T>(ctx, p, u_save, L->rank, L->scale, (const T*)dY, lddy, L->d_out, dB, accumulate, off, st)) != MLORA_OK)
    return s;
  if ((s = simt_grad<T>(ctx, p, ctx->ws_p, L->rank, nullptr, (const T*)x_save, L->d_in, L->d_in, dA, accumulate, ctx->drop,
                        st)) != MLORA_OK)
    return s;
  if (dX)
    s = simt_gemm<T, true>(ctx, (const T*)dY, lddy, (const T*)L->W, L->ldw, (const T*)L->A_all, ctx->ws_p, nullptr,
                           p->bwd, (T*)dX, lddx, Tft, L->d_in, L->d_out, L->rank, L->n_adapters, ctx->drop, st);
  return s;
}

}  // namespace

// ---- allocation-free forward ------------------------------------------------------------------
// Scratch for mlora_forward_noalloc: the rank-r intermediate of up to MLORA_NOALLOC_MAX_ROWS rows.
// It lives in the library image, so every device that loads the library carries these 256 KiB.
// In host code this name is only a handle; the device address is looked up once per device.
static __device__ __align__(256) float g_noalloc_scratch[MLORA_NOALLOC_MAX_ROWS * mlora::kMaxRank];

namespace {
float* g_noalloc_addr[kMaxDevices] = {};
std::mutex g_noalloc_mutex;

// Device address of the scratch on the current device (looked up on first use, then cached).
mlora_status_t noalloc_scratch(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MLORA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_addr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return MLORA_ERR_CUDA;
    }
    g_noalloc_addr[dev] = p;
  }
  *out = g_noalloc_addr[dev];
  return MLORA_OK;
}

template <typename T>
mlora_status_t forward_noalloc_t(const mlora_layer_t* L, const int32_t* row_adapter, int n_rows, const void* X,
                                 int64_t ldx, void* Y, int64_t ldy, float* scratch, cudaStream_t st) {
  const int64_t warps = (int64_t)n_rows * L->rank;
  const int blocks = (int)((warps * 32 + 255) / 256);
  // rank-r intermediate of every row (zeros for rows without an adapter, or with an id outside the layer's
  // adapter tables: the caller's device table has not been validated by anyone) -> scratch
  simt::shrink_kernel<T><<<blocks, 256, 0, st>>>((const T*)X, ldx, L->d_in, L->rank, (const T*)L->A_all, nullptr,
                                                 row_adapter, nullptr, scratch, (T*)nullptr, nullptr, 0, n_rows,
                                                 L->n_adapters, DropArgs{0, 0, 1.0f});
  if (cudaGetLastError() != cudaSuccess) return MLORA_ERR_CUDA;
  dim3 grid((L->d_out + 31) / 32, (n_rows + 31) / 32), block(32, 32);
  simt::gemm_lora_kernel<T, false><<<grid, block, 0, st>>>((const T*)X, ldx, (const T*)L->W, L->ldw,
                                                           (const T*)L->B_all, scratch, L->scale, row_adapter, (T*)Y,
                                                           ldy, n_rows, L->d_out, L->d_in, L->rank, L->n_adapters,
                                                           DropArgs{0, 0, 1.0f});
  return cudaGetLastError() == cudaSuccess ? MLORA_OK : MLORA_ERR_CUDA;
}
}  // namespace

// =============================================================================================
extern "C" {

mlora_status_t mlora_forward_noalloc(const mlora_layer_t* L, const int32_t* row_adapter, int32_t n_rows, const void* X,
                                     int64_t ldx, void* Y, int64_t ldy, void* cuda_stream) {
  if (!L || !L->W || !L->A_all || !L->B_all || !L->scale || n_rows < 0) return MLORA_ERR_INVALID_ARG;
  if (L->d_in <= 0 || L->d_out <= 0 || L->rank <= 0 || L->n_adapters <= 0 || L->ldw < L->d_out) return MLORA_ERR_INVALID_ARG;
  if (L->dtype != MLORA_F32 && L->dtype != MLORA_BF16) return MLORA_ERR_INVALID_ARG;
  if (n_rows > MLORA_NOALLOC_MAX_ROWS || L->rank > kMaxRank) return MLORA_ERR_UNSUPPORTED;
  if (n_rows == 0) return MLORA_OK;
  if (!row_adapter || !X || !Y || ldx < L->d_in || ldy < L->d_out) return MLORA_ERR_INVALID_ARG;
  float* scratch = nullptr;
  mlora_status_t s = noalloc_scratch(&scratch);
  if (s != MLORA_OK) return s;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (L->dtype == MLORA_F32) return forward_noalloc_t<float>(L, row_adapter, n_rows, X, ldx, Y, ldy, scratch, st);
  return forward_noalloc_t<__nv_bfloat16>(L, row_adapter, n_rows, X, ldx, Y, ldy, scratch, st);
}

const char* mlora_status_string(mlora_status_t s) {
  switch (s) {
    case MLORA_OK: return "ok";
    case MLORA_ERR_INVALID_ARG: return "invalid argument";
    case MLORA_ERR_SEGMENT_RANGE: return "segment outside the batch rows";
    case MLORA_ERR_SEGMENT_OVERLAP: return "segments overlap";
    case MLORA_ERR_ADAPTER_ID: return "adapter id out of range (or fine-tuning segment without adapter)";
    case MLORA_ERR_SAVE_CAPACITY: return "fine-tuning rows exceed the activation buffer capacity";
    case MLORA_ERR_UNSUPPORTED: return "shape, rank or alignment not supported";
    case MLORA_ERR_ARCH: return "no sm_100 CUDA device";
    case MLORA_ERR_CUDA: return "CUDA call failed";
    case MLORA_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case MLORA_CANCELLED: return "cancelled by the caller's flag";
  }
  return "unknown status";
}

mlora_status_t mlora_create(mlora_ctx** out, int device) {
  if (!out) return MLORA_ERR_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || n <= 0) { cudaGetLastError(); return MLORA_ERR_ARCH; }
  if (device < 0 || device >= n || device >= kMaxDevices) return MLORA_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MLORA_ERR_CUDA;
  if (prop.major != 10) return MLORA_ERR_ARCH;
  if (cudaSetDevice(device) != cudaSuccess) return MLORA_ERR_CUDA;
  mlora_ctx* c = new (std::nothrow) mlora_ctx();
  if (!c) return MLORA_ERR_INVALID_ARG;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !fn) {
    delete c;
    return MLORA_ERR_CUDA;
  }
  c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(&c->status_dev, sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&c->ws_splitk, kSplitKBytes) != cudaSuccess ||
      cudaMalloc(&c->ws_gpart, (size_t)c->sm_count * 4 * 65536) != cudaSuccess ||
      cudaMalloc(&c->ws_gcounters, (size_t)c->sm_count * sizeof(int32_t)) != cudaSuccess ||
      cudaMemset(c->ws_gcounters, 0, (size_t)c->sm_count * sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&c->ws_tc_counters, (size_t)kTcCounters * sizeof(int32_t)) != cudaSuccess ||
      cudaMemset(c->ws_tc_counters, 0, (size_t)kTcCounters * sizeof(int32_t)) != cudaSuccess ||
      cudaMemset(c->status_dev, 0, sizeof(int32_t)) != cudaSuccess) {
    cudaGetLastError();
    mlora_destroy(c);       // frees whatever was allocated
    return MLORA_ERR_CUDA;
  }
  *out = c;
  return MLORA_OK;
}

mlora_status_t mlora_profile_enable(mlora_ctx* c, int32_t max_records) {
  if (!c || max_records < 0) return MLORA_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return MLORA_ERR_CUDA;
  for (cudaEvent_t e : c->ev_start) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_stop) cudaEventDestroy(e);
  c->ev_start.clear(); c->ev_stop.clear(); c->ev_kind.clear(); c->ev_used = 0;
  for (int32_t i = 0; i < max_records; ++i) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess) return MLORA_ERR_CUDA;
    if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return MLORA_ERR_CUDA; }
    c->ev_start.push_back(a); c->ev_stop.push_back(b); c->ev_kind.push_back(0);
  }
  return MLORA_OK;
}

int32_t mlora_profile_collect(mlora_ctx* c, int32_t* kinds, float* ms, int32_t cap) {
  if (!c) return 0;
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  const int32_t n = c->ev_used;
  for (int32_t i = 0; i < n && i < cap; ++i) {
    float t = 0.f;
    cudaEventElapsedTime(&t, c->ev_start[i], c->ev_stop[i]);
    if (kinds) kinds[i] = c->ev_kind[i];
    if (ms) ms[i] = t;
  }
  c->ev_used = 0;
  return n;
}

void mlora_destroy(mlora_ctx* c) {
  if (!c) return;
  cudaSetDevice(c->device);
  for (cudaEvent_t e : c->ev_start) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_stop) cudaEventDestroy(e);
  cudaFree(c->status_dev);
  cudaFree(c->ws_p);
  cudaFree(c->ws_partial);
  cudaFree(c->ws_counters);
  cudaFree(c->ws_pbd);
  cudaFree(c->ws_splitk);
  cudaFree(c->ws_gpart);
  cudaFree(c->ws_gcounters);
  cudaFree(c->ws_tc_counters);
  for (void* r : c->retired) cudaFree(r);
  for (PlanBuf& b : c->plan_pool) free_plan_buf(b);
  delete c;
}

namespace {

constexpr int kPlanTables = 56;

// All device tables of a plan, packed; o[] receives each table's offset in 32-bit words.
void pack_plan(const HostPlan& h, BlobBuilder& b, size_t* o) {
  int n = 0;
  const RowSpace* rs[2] = {&h.fwd, &h.bwd};
  for (int i = 0; i < 2; ++i) {
    o[n++] = b.add(rs[i]->row_adapter); o[n++] = b.add(rs[i]->row_save); o[n++] = b.add(rs[i]->row_grp);
    o[n++] = b.add(rs[i]->tile_grp_off); o[n++] = b.add(rs[i]->grp_adapter); o[n++] = b.add(rs[i]->item_rows);
    o[n++] = b.add(rs[i]->row_grp2); o[n++] = b.add(rs[i]->tile2_grp_off); o[n++] = b.add(rs[i]->grp2_adapter);
    o[n++] = b.add(rs[i]->zero_rows2);
    o[n++] = b.add(rs[i]->item_save); o[n++] = b.add(rs[i]->item_start); o[n++] = b.add(rs[i]->item_desc);
    o[n++] = b.add(rs[i]->item_nrows); o[n++] = b.add(rs[i]->item_adapter);
    o[n++] = b.add(rs[i]->tcb_row0); o[n++] = b.add(rs[i]->tcb_nrows); o[n++] = b.add(rs[i]->tcb_adapter);
    o[n++] = b.add(rs[i]->grp2_col); o[n++] = b.add(rs[i]->grp2_width); o[n++] = b.add(rs[i]->tile2_cols);
    o[n++] = b.add(rs[i]->tile2_piece_off); o[n++] = b.add(rs[i]->piece_src);
    o[n++] = b.add(rs[i]->tcb_width);
  }
  o[n++] = b.add(h.slot_chunk_off); o[n++] = b.add(h.chunk_row0); o[n++] = b.add(h.chunk_nrows);
  o[n++] = b.add(h.ft_adapters);
  o[n++] = b.add(h.slot_blk_off); o[n++] = b.add(h.blk_row0); o[n++] = b.add(h.blk_nrows);
  o[n++] = b.add(h.slot_width);
}

// Words to reserve behind the plan's tables for unit lists: only row spaces whose 256-row tiles differ in
// their number of adapter groups can need one.
size_t sched_reserve(mlora_plan* p) {
  const RowSpace* rs[2] = {&p->h.fwd, &p->h.bwd};
  size_t words = 0;
  for (int i = 0; i < 2; ++i) {
    int32_t lo = 1 << 30, hi = 0;
    const std::vector<int32_t>& off = rs[i]->tile2_grp_off;
    for (size_t t = 0; t + 1 < off.size(); ++t) {
      const int32_t g = off[t + 1] - off[t];
      lo = g < lo ? g : lo; hi = g > hi ? g : hi;
    }
    p->sched[i].lc_spread = hi > lo ? hi - lo : 0;
    if (off.size() > 2 && hi - lo >= 2) words += (size_t)kSchedSlots * kSchedCap;
  }
  return words;
}
// Points the unit-list areas at the reserved words that start at word `at` of the blob, and their pinned mirrors at
// `mirror` (which holds the reserved words only; nullptr: no lists for this plan).
void bind_sched(mlora_plan* p, size_t at, int32_t* mirror) {
  const RowSpace* rs[2] = {&p->h.fwd, &p->h.bwd};
  DevRowSpace* ds[2] = {&p->fwd, &p->bwd};
  size_t m = 0;
  for (int i = 0; i < 2; ++i) {
    ds[i]->sched = &p->sched[i];
    if (mirror && rs[i]->tile2_grp_off.size() > 2 && p->sched[i].lc_spread >= 2) {
      p->sched[i].dev = p->blob + at + m;
      p->sched[i].mirror = mirror + m;
      m += (size_t)kSchedSlots * kSchedCap;
    }
  }
}

// Points the plan's table pointers into p->blob.
void bind_plan(mlora_plan* p, const size_t* o) {
  DevRowSpace* ds[2] = {&p->fwd, &p->bwd};
  int n = 0;
  for (int i = 0; i < 2; ++i) {
    ds[i]->row_adapter = p->blob + o[n++]; ds[i]->row_save = p->blob + o[n++]; ds[i]->row_grp = p->blob + o[n++];
    ds[i]->tile_grp_off = p->blob + o[n++]; ds[i]->grp_adapter = p->blob + o[n++]; ds[i]->item_rows = p->blob + o[n++];
    ds[i]->row_grp2 = p->blob + o[n++]; ds[i]->tile2_grp_off = p->blob + o[n++]; ds[i]->grp2_adapter = p->blob + o[n++];
    ds[i]->zero_rows2 = p->blob + o[n++];
    ds[i]->item_save = p->blob + o[n++]; ds[i]->item_start = p->blob + o[n++]; ds[i]->item_desc = p->blob + o[n++];
    ds[i]->item_nrows = p->blob + o[n++]; ds[i]->item_adapter = p->blob + o[n++];
    ds[i]->tcb_row0 = p->blob + o[n++]; ds[i]->tcb_nrows = p->blob + o[n++]; ds[i]->tcb_adapter = p->blob + o[n++];
    const bool ranked = !p->h.adapter_rank.empty();
    ds[i]->grp2_col = ranked ? p->blob + o[n] : nullptr; ++n;
    ds[i]->grp2_width = ranked ? p->blob + o[n] : nullptr; ++n;
    ds[i]->tile2_cols = ranked ? p->blob + o[n] : nullptr; ++n;
    ds[i]->tile2_piece_off = ranked ? p->blob + o[n] : nullptr; ++n;
    ds[i]->piece_src = ranked ? p->blob + o[n] : nullptr; ++n;
    ds[i]->tcb_width = ranked ? p->blob + o[n] : nullptr; ++n;
  }
  p->bwd.row_save = nullptr;       // the compact space has no save offsets
  p->slot_chunk_off = p->blob + o[n++]; p->chunk_row0 = p->blob + o[n++]; p->chunk_nrows = p->blob + o[n++];
  p->slot_adapter = p->blob + o[n++];
  p->slot_blk_off = p->blob + o[n++]; p->blk_row0 = p->blob + o[n++]; p->blk_nrows = p->blob + o[n++];
  p->slot_width = p->h.slot_width.empty() ? nullptr : p->blob + o[n]; ++n;
}

// Grows the context's workspaces to what this plan needs.  A workspace that is too small is REPLACED
// by a larger one (at least half as large again), never freed or moved: the old block stays allocated
// until mlora_destroy, so launches that already carry its address - kernels still queued, and above
// all kernels inside a captured CUDA graph - keep working on memory that is theirs.  In steady state
// nothing happens here.
mlora_status_t replace_workspace(mlora_ctx* ctx, void** ptr, size_t bytes, bool zero) {
  void* fresh = nullptr;
  if (cudaMalloc(&fresh, bytes) != cudaSuccess) { cudaGetLastError(); return MLORA_ERR_CUDA; }
  if (zero && cudaMemset(fresh, 0, bytes) != cudaSuccess) { cudaFree(fresh); return MLORA_ERR_CUDA; }
  if (*ptr) ctx->retired.push_back(*ptr);
  *ptr = fresh;
  return MLORA_OK;
}

mlora_status_t grow_workspaces(mlora_ctx* ctx, const HostPlan& h, int32_t n_rows) {
  mlora_status_t s;
  auto grown = [](int64_t need, int64_t have) { return need > have + have / 2 ? need : have + have / 2; };
  if (n_rows > ctx->ws_rows) {     // the rank-r workspace
    const int64_t rows = grown(n_rows, ctx->ws_rows);
    if ((s = replace_workspace(ctx, (void**)&ctx->ws_p, (size_t)rows * kMaxRank * sizeof(float), false)) != MLORA_OK) return s;
    if ((s = replace_workspace(ctx, (void**)&ctx->ws_tc_part, (size_t)(rows + 128 * ctx->sm_count) * kMaxRank * sizeof(float),
                               false)) != MLORA_OK) return s;
    ctx->ws_rows = rows;
  }
  const int64_t items = h.fwd.n_items() > h.bwd.n_items() ? h.fwd.n_items() : h.bwd.n_items();
  if (items + 4 * ctx->sm_count > ctx->ws_partial_items || items > ctx->ws_counter_items) {
    const int64_t it = grown(items, ctx->ws_counter_items);
    const int64_t part_items = it + 4 * ctx->sm_count;      // items * ksplit never exceeds this
    if ((s = replace_workspace(ctx, (void**)&ctx->ws_partial, (size_t)part_items * kItemRows * kMaxRank * sizeof(float), false)) != MLORA_OK ||
        (s = replace_workspace(ctx, (void**)&ctx->ws_counters, (size_t)(2 * it + 1) * sizeof(int32_t), true)) != MLORA_OK)
      return s;
    ctx->ws_partial_items = part_items; ctx->ws_counter_items = it;
  }
  const int64_t blocks = (int64_t)h.blk_row0.size();
  if (blocks > ctx->ws_pop_blocks && blocks <= kPopMaxBlocks) {      // beyond that the gradient kernel converts per tile
    const int64_t nb = grown(blocks, ctx->ws_pop_blocks) < kPopMaxBlocks ? grown(blocks, ctx->ws_pop_blocks) : kPopMaxBlocks;
    if ((s = replace_workspace(ctx, (void**)&ctx->ws_pop, (size_t)nb * 2 * 65536, false)) != MLORA_OK) return s;
    ctx->ws_pop_blocks = nb;
  }
  const int64_t groups = (int64_t)(h.fwd.grp2_adapter.size() > h.bwd.grp2_adapter.size() ? h.fwd.grp2_adapter.size()
                                                                                        : h.bwd.grp2_adapter.size());
  if (groups > ctx->ws_pbd_groups) {   // two chunk slots of [256][64] bf16 per adapter group of a tile
    const int64_t g = grown(groups, ctx->ws_pbd_groups);
    if ((s = replace_workspace(ctx, (void**)&ctx->ws_pbd, (size_t)g * 2 * 256 * 64 * sizeof(__nv_bfloat16), false)) != MLORA_OK) return s;
    ctx->ws_pbd_groups = g;
  }
  return MLORA_OK;
}

}  // namespace

mlora_status_t mlora_plan_create(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs, int32_t n_rows,
                                 int32_t n_adapters, mlora_plan** out) {
  return mlora_plan_create_ranked(ctx, segs, n_segs, n_rows, n_adapters, nullptr, out);
}

mlora_status_t mlora_plan_create_ranked(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs, int32_t n_rows,
                                        int32_t n_adapters, const int32_t* adapter_rank, mlora_plan** out) {
  if (!out) return MLORA_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx) {                          // host-only plan: tables for inspection, nothing on a device
    mlora_plan* p = new (std::nothrow) mlora_plan();
    if (!p) return MLORA_ERR_INVALID_ARG;
    const mlora_status_t s = build_plan(segs, n_segs, n_rows, n_adapters, p->h, adapter_rank);
    if (s != MLORA_OK) { delete p; return s; }
    *out = p;
    return MLORA_OK;
  }
  // With a context: the stream-ordered plan on the default stream, and the upload waited for.  The buffer pair
  // comes from (and mlora_plan_destroy returns it to) the context's pool, so that in steady state this call
  // makes no cudaMalloc / cudaMallocHost / cudaFree - each of them milliseconds when the driver has to map pages.
  mlora_status_t s = mlora_plan_create_ranked_async(ctx, segs, n_segs, n_rows, n_adapters, adapter_rank, nullptr, out);
  if (s != MLORA_OK) return s;
  if (cudaStreamSynchronize(nullptr) != cudaSuccess) {
    cudaGetLastError();
    mlora_plan_destroy(*out);
    *out = nullptr;
    return MLORA_ERR_CUDA;
  }
  return MLORA_OK;
}

mlora_status_t mlora_plan_create_async(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs, int32_t n_rows,
                                       int32_t n_adapters, void* cuda_stream, mlora_plan** out) {
  return mlora_plan_create_ranked_async(ctx, segs, n_segs, n_rows, n_adapters, nullptr, cuda_stream, out);
}

mlora_status_t mlora_plan_create_ranked_async(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs, int32_t n_rows,
                                              int32_t n_adapters, const int32_t* adapter_rank, void* cuda_stream,
                                              mlora_plan** out) {
  if (!out || !ctx) return MLORA_ERR_INVALID_ARG;
  *out = nullptr;
  mlora_plan* p = new (std::nothrow) mlora_plan();
  if (!p) return MLORA_ERR_INVALID_ARG;
  mlora_status_t s = build_plan(segs, n_segs, n_rows, n_adapters, p->h, adapter_rank);
  if (s != MLORA_OK) { delete p; return s; }
  p->ctx = ctx;
  if (cudaSetDevice(ctx->device) != cudaSuccess) { delete p; return MLORA_ERR_CUDA; }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  BlobBuilder b;
  size_t o[kPlanTables];
  pack_plan(p->h, b, o);
  const size_t tables = b.data.size();
  const size_t need = tables + sched_reserve(p);
  // a released buffer pair that is large enough and whose last user has passed its release point
  for (size_t i = 0; i < ctx->plan_pool.size(); ++i) {
    PlanBuf& c = ctx->plan_pool[i];
    if (c.cap >= need && cudaEventQuery(c.free_evt) == cudaSuccess) {
      p->buf = c;
      ctx->plan_pool[i] = ctx->plan_pool.back();
      ctx->plan_pool.pop_back();
      break;
    }
  }
  cudaGetLastError();                 // cudaEventQuery reports "not ready" through the error state
  if (!p->buf.dev) {
    size_t cap = 4096;
    while (cap < need) cap *= 2;
    if (cudaMalloc(&p->buf.dev, cap * sizeof(int32_t)) != cudaSuccess ||
        cudaMallocHost(&p->buf.pinned, cap * sizeof(int32_t)) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->buf.free_evt, cudaEventDisableTiming) != cudaSuccess) {
      free_plan_buf(p->buf); delete p; return MLORA_ERR_CUDA;
    }
    p->buf.cap = cap;
  }
  p->pooled = true;
  p->blob = p->buf.dev;
  std::memcpy(p->buf.pinned, b.data.data(), tables * sizeof(int32_t));
  if (cudaMemcpyAsync(p->blob, p->buf.pinned, tables * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess) {
    free_plan_buf(p->buf); delete p; return MLORA_ERR_CUDA;
  }
  bind_plan(p, o);
  bind_sched(p, tables, p->buf.pinned + tables);
  if ((s = grow_workspaces(ctx, p->h, n_rows)) != MLORA_OK) { free_plan_buf(p->buf); delete p; return s; }
  *out = p;
  return MLORA_OK;
}

mlora_status_t mlora_plan_release(mlora_plan* p, void* cuda_stream) {
  if (!p) return MLORA_OK;
  if (!p->pooled || !p->ctx) { mlora_plan_destroy(p); return MLORA_OK; }
  mlora_ctx* ctx = p->ctx;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return MLORA_ERR_CUDA;
  if (cudaEventRecord(p->buf.free_evt, reinterpret_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return MLORA_ERR_CUDA;
  if (ctx->plan_pool.size() < 64) ctx->plan_pool.push_back(p->buf);
  else free_plan_buf(p->buf);        // (frees wait for the device: only when far more plans are released than reused)
  delete p;
  return MLORA_OK;
}

void mlora_plan_destroy(mlora_plan* p) {
  if (!p) return;
  if (p->ctx) cudaSetDevice(p->ctx->device);
  if (p->pooled && p->ctx) {
    // wait for the device (whatever stream used the plan last), then the pair is free for the next plan
    const bool idle = cudaDeviceSynchronize() == cudaSuccess;
    if (!idle) cudaGetLastError();
    if (idle && p->ctx->plan_pool.size() < 64) p->ctx->plan_pool.push_back(p->buf);
    else free_plan_buf(p->buf);
  } else if (p->pooled) {
    free_plan_buf(p->buf);
  } else if (p->blob) {
    cudaFree(p->blob);
  }
  if (p->sched_pinned) cudaFreeHost(p->sched_pinned);
  delete p;
}

int32_t mlora_plan_rows(const mlora_plan* p) { return p ? p->h.n_rows : 0; }
int32_t mlora_plan_ft_rows(const mlora_plan* p) { return p ? p->h.ft_rows : 0; }
int32_t mlora_plan_ft_adapters(const mlora_plan* p, int32_t* ids, int32_t cap) {
  if (!p) return 0;
  const int32_t n = (int32_t)p->h.ft_adapters.size();
  for (int32_t i = 0; ids && i < n && i < cap; ++i) ids[i] = p->h.ft_adapters[i];
  return n;
}
int32_t mlora_plan_lowrank_columns(const mlora_plan* p, int32_t rank, int32_t* cols, int32_t cap) {
  if (!p) return 0;
  const RowSpace& rs = p->h.fwd;
  const int32_t tiles = (int32_t)rs.tile2_grp_off.size() - 1;
  for (int32_t t = 0; t < tiles && t < cap && cols; ++t)
    cols[t] = rs.tile2_cols.empty() ? (rs.tile2_grp_off[t + 1] - rs.tile2_grp_off[t]) * rank : rs.tile2_cols[t];
  return tiles < 0 ? 0 : tiles;
}

mlora_status_t mlora_plan_describe(const mlora_plan* p, int32_t* seg_save_offset, int32_t* row_adapter) {
  if (!p) return MLORA_ERR_INVALID_ARG;
  if (seg_save_offset) for (int32_t k = 0; k < p->h.n_segs; ++k) seg_save_offset[k] = p->h.seg_save_off[k];
  if (row_adapter) for (int32_t t = 0; t < p->h.n_rows; ++t) row_adapter[t] = p->h.fwd.row_adapter[t];
  return MLORA_OK;
}

mlora_status_t mlora_mixed_forward(mlora_ctx* ctx, const mlora_layer_t* L, const mlora_plan* p, const void* X,
                                   int64_t ldx, void* Y, int64_t ldy, void* x_save, float* u_save,
                                   int64_t save_row_base, int64_t save_capacity_rows, void* cuda_stream) {
  if (!ctx || !p || p->ctx != ctx || !p->blob) return MLORA_ERR_INVALID_ARG;
  mlora_status_t s = check_layer(L);
  if (s != MLORA_OK) return s;
  const HostPlan& h = p->h;
  if (h.n_adapters > L->n_adapters) return MLORA_ERR_ADAPTER_ID;
  if (h.n_rows == 0) return MLORA_OK;
  if (!X || !Y || ldx < L->d_in || ldy < L->d_out) return MLORA_ERR_INVALID_ARG;
  if (save_row_base < 0 || save_capacity_rows < 0) return MLORA_ERR_INVALID_ARG;
  if (h.ft_rows > 0) {
    if (save_row_base + h.ft_rows > save_capacity_rows) return MLORA_ERR_SAVE_CAPACITY;
    if (!u_save) return MLORA_ERR_INVALID_ARG;
  }
  if (h.n_rows > ctx->ws_rows || !ranked_plan_fits(h, L)) return MLORA_ERR_INVALID_ARG;
  // the tensor maps are encoded through the driver API, which needs this device's context current on the
  // calling thread (a framework's worker threads do not always have one)
  if (cudaSetDevice(ctx->device) != cudaSuccess) return MLORA_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (L->dtype == MLORA_F32)
    return forward_simt<float>(ctx, L, p, X, ldx, Y, ldy, x_save, u_save, save_row_base, st);
  if (ldx % 8 || ldy % 8 || !aligned16(X) || !aligned16(Y) || (x_save && !aligned16(x_save))) return MLORA_ERR_UNSUPPORTED;
  if (ctx->gemm_path == 1)
    return forward_simt<__nv_bfloat16>(ctx, L, p, X, ldx, Y, ldy, x_save, u_save, save_row_base, st);

  if (ctx->drop.thr != 0 && h.ft_rows > 0 && ctx->shrink_path != 0 && L->rank <= 64) return MLORA_ERR_UNSUPPORTED;
  ShrinkArgs sa;
  sa.In = (const __nv_bfloat16*)X; sa.ld_in = ldx; sa.D = L->d_in;
  sa.P_all = (const __nv_bfloat16*)L->A_all; sa.scale = nullptr; sa.Out = ctx->ws_p;
  sa.item_rows = p->fwd.item_rows; sa.item_start = p->fwd.item_start; sa.item_nrows = p->fwd.item_nrows;
  sa.item_adapter = p->fwd.item_adapter; sa.item_save = p->fwd.item_save;
  sa.pbd = PbdArgs{ctx->gemm_pairs ? ctx->ws_pbd : nullptr, p->fwd.row_grp2, p->fwd.tile2_grp_off, L->scale,
                   p->fwd.zero_rows2, (int32_t)h.fwd.zero_rows2.size()};
  set_ranked(sa.pbd, p->fwd);
  sa.x_save = (__nv_bfloat16*)x_save; sa.u_save = u_save; sa.save_base = save_row_base;
  sa.save_cap = save_capacity_rows;
  // rank >= kTcShrinkMinRank (every rank under kernel variant 6): the tcgen05 shrink and its finish kernel
  const bool tc_shrink = ctx->shrink_path == 0 && ctx->drop.thr == 0 && !h.fwd.tcb_row0.empty() &&
                         (L->rank >= kTcShrinkMinRank || ctx->grad_mode == 2) && shrink_tc_fits(ctx, h.fwd, h.n_rows, L->d_in, L->rank);
  if (tc_shrink) {
    stc::FinArgs fa = {};
    fa.scale = nullptr; fa.Out = ctx->ws_p; fa.pbd = sa.pbd;
    fa.row_save = h.ft_rows > 0 ? p->fwd.row_save : nullptr; fa.u_save = u_save;
    fa.X = (const __nv_bfloat16*)X; fa.ldx = ldx; fa.x_save = (__nv_bfloat16*)x_save; fa.save_base = save_row_base; fa.D = L->d_in;
    s = launch_shrink_tc_any(ctx, L->rank, h.fwd, p->fwd, X, ldx, h.n_rows, L->d_in, L->A_all, L->n_adapters, fa, st);
  } else {
    s = launch_shrink(ctx, L->rank, sa, h.fwd.n_items(), p->fwd.item_desc, h.n_rows, L->n_adapters, st);
  }
  if (s != MLORA_OK) return s;
  return gemm_bf16<false>(ctx, L, h.fwd, p->fwd, X, ldx, Y, ldy, L->B_all, ctx->ws_p, L->scale, h.n_rows, L->d_out,
                          L->d_in, st);
}

mlora_status_t mlora_backward(mlora_ctx* ctx, const mlora_layer_t* L, const mlora_plan* p, const void* dY, int64_t lddy,
                              const void* x_save, const float* u_save, float* dA, float* dB, void* dX, int64_t lddx,
                              int32_t accumulate, void* cuda_stream) {
  if (!ctx || !p || p->ctx != ctx || !p->blob) return MLORA_ERR_INVALID_ARG;
  mlora_status_t s = check_layer(L);
  if (s != MLORA_OK) return s;
  const HostPlan& h = p->h;
  if (h.n_adapters > L->n_adapters) return MLORA_ERR_ADAPTER_ID;
  if (h.ft_rows == 0) return MLORA_OK;
  if (!dY || !x_save || !u_save || !dA || !dB || lddy < L->d_out || (dX && lddx < L->d_in)) return MLORA_ERR_INVALID_ARG;
  if (!ranked_plan_fits(h, L)) return MLORA_ERR_INVALID_ARG;
  // the tensor maps are encoded through the driver API, which needs this device's context current on the
  // calling thread (a framework's worker threads do not always have one)
  if (cudaSetDevice(ctx->device) != cudaSuccess) return MLORA_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (L->dtype == MLORA_F32)
    return backward_simt<float>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, dX, lddx, accumulate, st);
  if (lddy % 8 || (dX && lddx % 8) || !aligned16(dY) || !aligned16(x_save) || (dX && !aligned16(dX)) ||
      !aligned16(dA) || !aligned16(dB) || !aligned16(u_save))
    return MLORA_ERR_UNSUPPORTED;
  if (ctx->gemm_path == 1)
    return backward_simt<__nv_bfloat16>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, dX, lddx, accumulate, st);

  const int n_slots = (int)h.ft_adapters.size();
  const bool dropping = ctx->drop.thr != 0;
  if (dropping && ctx->shrink_path != 0 && L->rank <= 64) return MLORA_ERR_UNSUPPORTED;
  ShrinkArgs sa;                     // V = s dY B^T
  sa.In = (const __nv_bfloat16*)dY; sa.ld_in = lddy; sa.D = L->d_out;
  sa.P_all = (const __nv_bfloat16*)L->B_all; sa.scale = L->scale; sa.Out = ctx->ws_p;
  sa.item_rows = p->bwd.item_rows; sa.item_start = p->bwd.item_start; sa.item_nrows = p->bwd.item_nrows;
  sa.pbd = PbdArgs{(ctx->gemm_pairs && dX && !dropping) ? ctx->ws_pbd : nullptr, p->bwd.row_grp2, p->bwd.tile2_grp_off, nullptr,
                   p->bwd.zero_rows2, (int32_t)h.bwd.zero_rows2.size()};
  set_ranked(sa.pbd, p->bwd);
  sa.item_adapter = p->bwd.item_adapter; sa.item_save = nullptr; sa.x_save = nullptr; sa.u_save = nullptr; sa.save_base = 0; sa.save_cap = 0;
  // V on the tcgen05 shrink from rank kTcShrinkMinRank (every rank under kernel variant 6), else on the mma.sync kernels
  const bool tc_v = ctx->shrink_path == 0 && (L->rank >= kTcShrinkMinRank || ctx->grad_mode == 2) &&
                    shrink_tc_fits(ctx, h.bwd, h.ft_rows, L->d_out, L->rank);
  if (tc_v) {
    stc::FinArgs fa = {};
    fa.scale = L->scale; fa.Out = ctx->ws_p; fa.pbd = sa.pbd;
    s = launch_shrink_tc_any(ctx, L->rank, h.bwd, p->bwd, dY, lddy, h.ft_rows, L->d_out, L->B_all, L->n_adapters, fa, st);
  } else {
    s = launch_shrink(ctx, L->rank, sa, h.bwd.n_items(), p->bwd.item_desc, h.ft_rows, L->n_adapters, st);
  }
  if (s != MLORA_OK) return s;

  GradArgs ga;                       // dB = (s U)^T dY
  ga.P = u_save; ga.R = L->rank; ga.scale = L->scale; ga.Q = (const __nv_bfloat16*)dY; ga.ldq = lddy; ga.D = L->d_out;
  ga.G = dB; ga.slot_chunk_off = p->slot_chunk_off; ga.chunk_row0 = p->chunk_row0; ga.chunk_nrows = p->chunk_nrows;
  ga.slot_adapter = p->slot_adapter; ga.accumulate = accumulate;
  GradArgs gA = ga;                  // dA = V^T X
  gA.P = ctx->ws_p; gA.scale = nullptr; gA.Q = (const __nv_bfloat16*)x_save; gA.ldq = L->d_in; gA.D = L->d_in; gA.G = dA;
  // both gradients on the tensor-core kernel where it is the faster one (V is in the workspace by now)
  bool tc_grad = false;
  if (ctx->grad_mode != 1 && ctx->shrink_path == 0 && !dropping && (ctx->grad_mode == 2 || L->rank >= kTcGradMinRank)) {
    switch (L->rank) {
      case 8: tc_grad = grad_tc_fits<8>(L, p); break;
      case 16: tc_grad = grad_tc_fits<16>(L, p); break;
      case 32: tc_grad = grad_tc_fits<32>(L, p); break;
      case 64: tc_grad = grad_tc_fits<64>(L, p); break;
      case 128: tc_grad = grad_tc_fits<128>(L, p); break;
    }
  }
  if (tc_grad) {
    switch (L->rank) {
      case 8: s = launch_grad_tc<8>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, accumulate, st); break;
      case 16: s = launch_grad_tc<16>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, accumulate, st); break;
      case 32: s = launch_grad_tc<32>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, accumulate, st); break;
      case 64: s = launch_grad_tc<64>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, accumulate, st); break;
      default: s = launch_grad_tc<128>(ctx, L, p, dY, lddy, x_save, u_save, dA, dB, accumulate, st); break;
    }
    if (s != MLORA_OK || !dX) return s;
    return gemm_bf16<true>(ctx, L, h.bwd, p->bwd, dY, lddy, dX, lddx, L->A_all, ctx->ws_p, nullptr, h.ft_rows, L->d_in,
                           L->d_out, st);
  }
  if (ctx->shrink_path == 0 && L->rank <= 64) {      // both gradients in one launch of the streaming kernel
    s = L->rank <= 16 ? launch_grad_stream2<1>(ctx, p, ga, gA, n_slots, h.ft_rows, st)
        : L->rank <= 32 ? launch_grad_stream2<2>(ctx, p, ga, gA, n_slots, h.ft_rows, st)
                        : launch_grad_stream2<4>(ctx, p, ga, gA, n_slots, h.ft_rows, st);
    if (s != MLORA_OK) return s;
    if (!dX) return MLORA_OK;
    if (dropping) {   // the mask acts on the low-rank term per element: base product first, then the masked expand
      if ((s = gemm_bf16<true>(ctx, L, h.bwd, p->bwd, dY, lddy, dX, lddx, L->A_all, ctx->ws_p, nullptr, h.ft_rows,
                               L->d_in, L->d_out, st, false)) != MLORA_OK)
        return s;
      return launch_expand_mask(ctx, L, p->bwd, dX, lddx, h.ft_rows, st);
    }
    return gemm_bf16<true>(ctx, L, h.bwd, p->bwd, dY, lddy, dX, lddx, L->A_all, ctx->ws_p, nullptr, h.ft_rows, L->d_in,
                           L->d_out, st);
  }
  if ((s = launch_grad(ctx, p, ga, n_slots, h.ft_rows, st)) != MLORA_OK) return s;
  ga.P = ctx->ws_p; ga.scale = nullptr; ga.Q = (const __nv_bfloat16*)x_save; ga.ldq = L->d_in; ga.D = L->d_in;
  ga.G = dA;                         // dA = V^T X (with dropout: the kept elements of X, V counted 1 / (1 - p) times)
  if (dropping) ga.drop = ctx->drop;
  if ((s = launch_grad(ctx, p, ga, n_slots, h.ft_rows, st)) != MLORA_OK) return s;
  if (!dX) return MLORA_OK;
  if (dropping) {   // the mask acts on the low-rank term per element: base product first, then the masked expand
    if ((s = gemm_bf16<true>(ctx, L, h.bwd, p->bwd, dY, lddy, dX, lddx, L->A_all, ctx->ws_p, nullptr, h.ft_rows, L->d_in,
                             L->d_out, st, false)) != MLORA_OK)
      return s;
    return launch_expand_mask(ctx, L, p->bwd, dX, lddx, h.ft_rows, st);
  }
  return gemm_bf16<true>(ctx, L, h.bwd, p->bwd, dY, lddy, dX, lddx, L->A_all, ctx->ws_p, nullptr, h.ft_rows, L->d_in,
                         L->d_out, st);
}

mlora_status_t mlora_adamw_update(mlora_ctx* ctx, const mlora_layer_t* L, const mlora_plan* p, const float* dA,
                                  const float* dB, float* wA, float* wB, float* mA, float* vA, float* mB, float* vB,
                                  const mlora_adamw_t* hp, void* cuda_stream) {
  if (!ctx || !p || p->ctx != ctx || !p->blob || !hp) return MLORA_ERR_INVALID_ARG;
  mlora_status_t s = check_layer(L);
  if (s != MLORA_OK) return s;
  const HostPlan& h = p->h;
  if (h.n_adapters > L->n_adapters) return MLORA_ERR_ADAPTER_ID;
  if (hp->step < 1 || !(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f))
    return MLORA_ERR_INVALID_ARG;
  const int n_slots = (int)h.ft_adapters.size();
  if (n_slots == 0) return MLORA_OK;
  if (!dA || !dB || !wA || !wB || !mA || !vA || !mB || !vB) return MLORA_ERR_INVALID_ARG;
  if (L->d_in % 4 || L->d_out % 4) return MLORA_ERR_UNSUPPORTED;
  simt::AdamwArgs a;
  a.side[0] = simt::AdamwSide{dA, wA, mA, vA, const_cast<void*>(L->A_all), L->d_in};
  a.side[1] = simt::AdamwSide{dB, wB, mB, vB, const_cast<void*>(L->B_all), L->d_out};
  a.slot_adapter = p->slot_adapter; a.n_slots = n_slots; a.R = L->rank;
  a.lr = hp->lr; a.beta1 = hp->beta1; a.beta2 = hp->beta2; a.eps = hp->eps; a.wd = hp->weight_decay;
  a.inv_bc1 = (float)(1.0 / (1.0 - pow((double)hp->beta1, (double)hp->step)));
  a.inv_bc2 = (float)(1.0 / (1.0 - pow((double)hp->beta2, (double)hp->step)));
  if (cancelled(ctx)) return MLORA_CANCELLED;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return MLORA_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int64_t widest = (int64_t)n_slots * L->rank * (L->d_in > L->d_out ? L->d_in : L->d_out) / 4;
  int blocks = (int)((widest + 255) / 256);
  blocks = blocks < 4 * ctx->sm_count ? blocks : 4 * ctx->sm_count;
  LaunchScope scope(ctx, st, KIND_ADAMW);
  if (L->dtype == MLORA_F32) simt::adamw_kernel<float><<<dim3(blocks, 2), 256, 0, st>>>(a);
  else simt::adamw_kernel<__nv_bfloat16><<<dim3(blocks, 2), 256, 0, st>>>(a);
  return scope.done();
}

mlora_status_t mlora_poll_status(mlora_ctx* ctx, void* cuda_stream) {
  if (!ctx) return MLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int32_t v = 0;
  if (cudaMemcpyAsync(&v, ctx->status_dev, sizeof(v), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MLORA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MLORA_ERR_CUDA;
  if (v != 0) {
    // A kernel that gave up may have left the arrival counters of split work items partly counted (only a
    // launch that runs to its end puts them back to zero), so they are cleared together with the word.
    cudaMemsetAsync(ctx->status_dev, 0, sizeof(v), st);
    if (ctx->ws_counters) cudaMemsetAsync(ctx->ws_counters, 0, (size_t)(2 * ctx->ws_counter_items + 1) * sizeof(int32_t), st);
    cudaMemsetAsync(ctx->ws_gcounters, 0, (size_t)ctx->sm_count * sizeof(int32_t), st);
    cudaMemsetAsync(ctx->ws_tc_counters, 0, (size_t)kTcCounters * sizeof(int32_t), st);
    cudaStreamSynchronize(st);
  }
  return (mlora_status_t)v;
}

mlora_status_t mlora_selftest_timeout(mlora_ctx* ctx, uint32_t polls, void* cuda_stream) {
  if (!ctx || polls == 0 || polls > (1u << 20)) return MLORA_ERR_INVALID_ARG;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return MLORA_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  LaunchScope scope(ctx, st, KIND_SIMT);
  wait_selftest_kernel<<<1, 64, 0, st>>>(ctx->status_dev, polls);
  return scope.done();
}

mlora_status_t mlora_set_cancel_flag(mlora_ctx* ctx, const volatile int32_t* host_flag) {
  if (!ctx) return MLORA_ERR_INVALID_ARG;
  ctx->cancel = host_flag;
  return MLORA_OK;
}

mlora_status_t mlora_set_dropout(mlora_ctx* ctx, double p, uint64_t seed) {
  if (!ctx || !(p >= 0.0 && p < 1.0)) return MLORA_ERR_INVALID_ARG;
  ctx->drop.seed = seed;
  ctx->drop.thr = (uint32_t)std::nearbyint(p * 65536.0);      // ties to even, as the oracle's rounding
  ctx->drop.keep_scale = (float)(1.0 / (1.0 - p));
  return MLORA_OK;
}

int64_t mlora_launch_count(const mlora_ctx* ctx) { return ctx ? ctx->launches : 0; }

mlora_status_t mlora_set_gemm_path(mlora_ctx* ctx, int32_t path) {
  if (!ctx || path < 0 || path > 7) return MLORA_ERR_INVALID_ARG;
  ctx->gemm_path = path == 1 ? 1 : 0;
  ctx->shrink_path = path == 2 ? 1 : 0;
  ctx->gemm_pairs = path == 3 ? 0 : 1;
  ctx->no_split_k = path == 4 ? 1 : 0;
  ctx->no_unit_lists = path == 7 ? 1 : 0;
  ctx->grad_mode = path == 5 ? 1 : (path == 6 ? 2 : 0);
  return MLORA_OK;
}

// ---- layer pieces around the projections (mlora_layer_ops.h) ----------------------------------
static inline mlora_status_t launched() {
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? MLORA_OK : cuda_failure("kernel launch", cudaGetErrorString(e));
}
static inline int ew_blocks(int64_t n8) {
  const int64_t b = (n8 + 255) / 256;
  return (int)(b < 148 * 8 ? (b < 1 ? 1 : b) : 148 * 8);
}

mlora_status_t mlora_rmsnorm_forward(const void* x, int64_t ldx, const float* gain, void* y, int64_t ldy,
                                     int32_t n_rows, int32_t d, float eps, void* cuda_stream) {
  if (!x || !gain || !y || n_rows < 0 || d <= 0 || ldx < d || ldy < d) return MLORA_ERR_INVALID_ARG;
  if (d % 8 || ldx % 8 || ldy % 8 || !aligned16(x) || !aligned16(y) || !aligned16(gain)) return MLORA_ERR_UNSUPPORTED;
  if (n_rows == 0) return MLORA_OK;
  glue::rmsnorm_fwd_kernel<<<n_rows, 128, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      (const __nv_bfloat16*)x, ldx, gain, (__nv_bfloat16*)y, ldy, d, eps);
  return launched();
}

mlora_status_t mlora_rmsnorm_backward(const void* x, int64_t ldx, const float* gain, const void* dy, int64_t lddy,
                                      void* dx, int64_t lddx, int32_t n_rows, int32_t d, float eps, void* cuda_stream) {
  if (!x || !gain || !dy || !dx || n_rows < 0 || d <= 0 || ldx < d || lddy < d || lddx < d) return MLORA_ERR_INVALID_ARG;
  if (d % 8 || ldx % 8 || lddy % 8 || lddx % 8 || !aligned16(x) || !aligned16(dy) || !aligned16(dx) || !aligned16(gain))
    return MLORA_ERR_UNSUPPORTED;
  if (n_rows == 0) return MLORA_OK;
  glue::rmsnorm_bwd_kernel<<<n_rows, 128, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      (const __nv_bfloat16*)x, ldx, gain, (const __nv_bfloat16*)dy, lddy, (__nv_bfloat16*)dx, lddx, d, eps);
  return launched();
}

mlora_status_t mlora_rope(const void* x, int64_t ldx, void* y, int64_t ldy, const int32_t* pos, int32_t n_rows,
                          int32_t n_heads, int32_t d_head, float theta, int32_t transpose, void* cuda_stream) {
  if (!x || !y || !pos || n_rows < 0 || n_heads <= 0 || d_head <= 0 || !(theta > 0.f)) return MLORA_ERR_INVALID_ARG;
  if (ldx < (int64_t)n_heads * d_head || ldy < (int64_t)n_heads * d_head) return MLORA_ERR_INVALID_ARG;
  if (d_head % 16 || ldx % 8 || ldy % 8 || !aligned16(x) || !aligned16(y)) return MLORA_ERR_UNSUPPORTED;
  if (n_rows == 0) return MLORA_OK;
  glue::rope_kernel<<<n_rows, 128, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      (const __nv_bfloat16*)x, ldx, (__nv_bfloat16*)y, ldy, pos, n_heads, d_head, log2f(theta), transpose ? -1.0f : 1.0f);
  return launched();
}

mlora_status_t mlora_swiglu_forward(const void* g, const void* u, void* m, int64_t n, void* cuda_stream) {
  if (!g || !u || !m || n < 0) return MLORA_ERR_INVALID_ARG;
  if (n % 8 || !aligned16(g) || !aligned16(u) || !aligned16(m)) return MLORA_ERR_UNSUPPORTED;
  if (n == 0) return MLORA_OK;
  glue::swiglu_fwd_kernel<<<ew_blocks(n / 8), 256, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      (const __nv_bfloat16*)g, (const __nv_bfloat16*)u, (__nv_bfloat16*)m, n / 8);
  return launched();
}

mlora_status_t mlora_swiglu_backward(const void* g, const void* u, const void* dm, void* dg, void* du, int64_t n,
                                     void* cuda_stream) {
  if (!g || !u || !dm || !dg || !du || n < 0) return MLORA_ERR_INVALID_ARG;
  if (n % 8 || !aligned16(g) || !aligned16(u) || !aligned16(dm) || !aligned16(dg) || !aligned16(du)) return MLORA_ERR_UNSUPPORTED;
  if (n == 0) return MLORA_OK;
  glue::swiglu_bwd_kernel<<<ew_blocks(n / 8), 256, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      (const __nv_bfloat16*)g, (const __nv_bfloat16*)u, (const __nv_bfloat16*)dm, (__nv_bfloat16*)dg, (__nv_bfloat16*)du, n / 8);
  return launched();
}

mlora_status_t mlora_add(const void* a, const void* b, void* out, int64_t n, void* cuda_stream) {
  if (!a || !b || !out || n < 0) return MLORA_ERR_INVALID_ARG;
  if (n % 8 || !aligned16(a) || !aligned16(b) || !aligned16(out)) return MLORA_ERR_UNSUPPORTED;
  if (n == 0) return MLORA_OK;
  glue::add_kernel<<<ew_blocks(n / 8), 256, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      (const __nv_bfloat16*)a, (const __nv_bfloat16*)b, (__nv_bfloat16*)out, n / 8);
  return launched();
}

}  // extern "C"

// Head size 128: the tcgen05 kernels.  The layer pieces have no context object, so the tensor-map
// encoder is looked up once per process here (only that entry of the object is used).
static mlora_ctx* layer_ops_encoder() {
  // function-local statics: the language runs this initialisation once, under its own lock
  static mlora_ctx enc;
  static bool ok = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess ||
        qr != cudaDriverEntryPointSuccess || !fn)
      return false;
    enc.encode = reinterpret_cast<EncodeTiledFn>(fn);
    return true;
  }();
  return ok ? &enc : nullptr;
}

template <typename Kern>
static mlora_status_t attn_tc_smem(Kern kern, uint32_t bytes, bool* done_dev) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MLORA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_attr_mutex);
  if (!done_dev[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return MLORA_ERR_CUDA;
    done_dev[dev] = true;
  }
  return MLORA_OK;
}

static mlora_status_t attention_forward_tc(const void* q, int64_t ldq, const void* k, int64_t ldk, const void* v,
                                           int64_t ldv, void* o, int64_t ldo, float* lse, const int32_t* seq_start,
                                           int32_t n_rows, int32_t n_heads, int32_t n_kv, cudaStream_t st) {
  mlora_ctx* enc = layer_ops_encoder();
  if (!enc) return MLORA_ERR_CUDA;
  static bool attr_dev[kMaxDevices] = {};
  mlora_status_t s;
  if ((s = attn_tc_smem(attn_tc::forward_kernel, attn_tc::SMEM_BYTES, attr_dev)) != MLORA_OK) return s;
  CUtensorMap tQ, tK, tV;
  if ((s = make_tmap_bf16(enc, &tQ, q, (uint64_t)n_heads * 128, n_rows, ldq, 64, 128)) != MLORA_OK) return s;
  if ((s = make_tmap_bf16(enc, &tK, k, (uint64_t)n_kv * 128, n_rows, ldk, 64, 128)) != MLORA_OK) return s;
  if ((s = make_tmap_bf16_blocked(enc, &tV, v, n_rows, (uint64_t)n_kv * 128, ldv, 64, 2)) != MLORA_OK) return s;
  attn_tc::Args a{(__nv_bfloat16*)o, ldo, lse, seq_start, n_rows, n_heads, n_kv, 1.4426950408889634f / sqrtf(128.0f)};
  attn_tc::forward_kernel<<<dim3((n_rows + 127) / 128, n_heads), attn_tc::FWD_THREADS, attn_tc::SMEM_BYTES, st>>>(tQ, tK, tV, a);
  return launched();
}

static mlora_status_t attention_backward_tc(const void* q, int64_t ldq, const void* k, int64_t ldk, const void* v, int64_t ldv,
                                            const void* o, int64_t ldo, const float* lse, const void* dO, int64_t lddo,
                                            void* dq, int64_t lddq, void* dk, int64_t lddk, void* dv, int64_t lddv,
                                            const int32_t* seq_start, const int32_t* seq_end, int32_t n_rows,
                                            int32_t n_heads, int32_t n_kv, cudaStream_t st) {
  mlora_ctx* enc = layer_ops_encoder();
  if (!enc) return MLORA_ERR_CUDA;
  static bool attr_dq[kMaxDevices] = {}, attr_dkv[kMaxDevices] = {};
  mlora_status_t s;
  if ((s = attn_tc_smem(attn_tc::backward_dq_kernel, attn_tc::DQ_SMEM_BYTES, attr_dq)) != MLORA_OK) return s;
  if ((s = attn_tc_smem(attn_tc::backward_dkv_kernel, attn_tc::DKV_SMEM_BYTES, attr_dkv)) != MLORA_OK) return s;
  CUtensorMap tQ, tdO, tO, tK, tV;       // all [rows][64-column] boxes of 128 rows
  if ((s = make_tmap_bf16(enc, &tQ, q, (uint64_t)n_heads * 128, n_rows, ldq, 64, 128)) != MLORA_OK) return s;
  if ((s = make_tmap_bf16(enc, &tdO, dO, (uint64_t)n_heads * 128, n_rows, lddo, 64, 128)) != MLORA_OK) return s;
  if ((s = make_tmap_bf16(enc, &tO, o, (uint64_t)n_heads * 128, n_rows, ldo, 64, 128)) != MLORA_OK) return s;
  if ((s = make_tmap_bf16(enc, &tK, k, (uint64_t)n_kv * 128, n_rows, ldk, 64, 128)) != MLORA_OK) return s;
  if ((s = make_tmap_bf16(enc, &tV, v, (uint64_t)n_kv * 128, n_rows, ldv, 64, 128)) != MLORA_OK) return s;
  const float scale = 1.0f / sqrtf(128.0f);
  attn_tc::BwdArgs a{(const __nv_bfloat16*)o, ldo, (const __nv_bfloat16*)dO, lddo, lse, seq_start, seq_end,
                     (__nv_bfloat16*)dq, lddq, (__nv_bfloat16*)dk, lddk, (__nv_bfloat16*)dv, lddv,
                     n_rows, n_heads, n_kv, scale, scale * 1.4426950408889634f};
  const int tiles = (n_rows + 127) / 128;
  attn_tc::backward_dq_kernel<<<dim3(tiles, n_heads), attn_tc::THREADS, attn_tc::DQ_SMEM_BYTES, st>>>(tQ, tdO, tK, tV, a);
  if ((s = launched()) != MLORA_OK) return s;
  attn_tc::backward_dkv_kernel<<<dim3(tiles, n_kv), attn_tc::THREADS, attn_tc::DKV_SMEM_BYTES, st>>>(tQ, tdO, tO, tK, tV, a);
  return launched();
}

extern "C" {

mlora_status_t mlora_attention_forward(const void* q, int64_t ldq, const void* k, int64_t ldk, const void* v, int64_t ldv,
                                       void* o, int64_t ldo, float* lse, const int32_t* seq_start, const int32_t* seq_end,
                                       int32_t n_rows, int32_t n_heads, int32_t n_kv, int32_t d_head, void* cuda_stream) {
  if (!q || !k || !v || !o || !lse || !seq_start || !seq_end || n_rows < 0 || n_heads <= 0 || n_kv <= 0)
    return MLORA_ERR_INVALID_ARG;
  if ((d_head != 64 && d_head != 128) || n_heads % n_kv) return MLORA_ERR_UNSUPPORTED;
  if (ldq % 8 || ldk % 8 || ldv % 8 || ldo % 8 || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o))
    return MLORA_ERR_UNSUPPORTED;
  if (n_rows == 0) return MLORA_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (d_head == 128) return attention_forward_tc(q, ldq, k, ldk, v, ldv, o, ldo, lse, seq_start, n_rows, n_heads, n_kv, st);
  attn::AttnArgs a{(const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, ldq, ldk, ldv,
                   seq_start, seq_end, n_rows, n_heads, n_kv, 1.0f / sqrtf((float)d_head)};
  const int blocks = (int)(((int64_t)n_rows * n_heads + 7) / 8);
  attn::forward_kernel<16><<<blocks, 256, 0, st>>>(a, (__nv_bfloat16*)o, ldo, lse);
  return launched();
}

mlora_status_t mlora_layer_ops_poll_status(void* cuda_stream) {
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return MLORA_ERR_CUDA;
  int32_t v = 0;
  if (cudaMemcpyFromSymbol(&v, attn_tc::g_status, sizeof v) != cudaSuccess) return MLORA_ERR_CUDA;
  if (v != 0) {
    const int32_t zero = 0;
    if (cudaMemcpyToSymbol(attn_tc::g_status, &zero, sizeof zero) != cudaSuccess) return MLORA_ERR_CUDA;
  }
  return (mlora_status_t)v;
}

mlora_status_t mlora_attention_backward(const void* q, int64_t ldq, const void* k, int64_t ldk, const void* v, int64_t ldv,
                                        const void* o, int64_t ldo, const float* lse, const void* dO, int64_t lddo,
                                        void* dq, int64_t lddq, void* dk, int64_t lddk, void* dv, int64_t lddv,
                                        const int32_t* seq_start, const int32_t* seq_end, int32_t n_rows,
                                        int32_t n_heads, int32_t n_kv, int32_t d_head, void* cuda_stream) {
  if (!q || !k || !v || !o || !lse || !dO || !dq || !dk || !dv || !seq_start || !seq_end || n_rows < 0 || n_heads <= 0 ||
      n_kv <= 0)
    return MLORA_ERR_INVALID_ARG;
  if ((d_head != 64 && d_head != 128) || n_heads % n_kv) return MLORA_ERR_UNSUPPORTED;
  if (ldq % 8 || ldk % 8 || ldv % 8 || ldo % 8 || lddo % 8 || lddq % 8 || lddk % 8 || lddv % 8 || !aligned16(q) ||
      !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(dO) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv))
    return MLORA_ERR_UNSUPPORTED;
  if (n_rows == 0) return MLORA_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (d_head == 128)
    return attention_backward_tc(q, ldq, k, ldk, v, ldv, o, ldo, lse, dO, lddo, dq, lddq, dk, lddk, dv, lddv, seq_start,
                                 seq_end, n_rows, n_heads, n_kv, st);
  attn::AttnArgs a{(const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, ldq, ldk, ldv,
                   seq_start, seq_end, n_rows, n_heads, n_kv, 1.0f / sqrtf((float)d_head)};
  const int bq = (int)(((int64_t)n_rows * n_heads + 7) / 8), bk = (int)(((int64_t)n_rows * n_kv + 7) / 8);
  {
    attn::backward_dq_kernel<16><<<bq, 256, 0, st>>>(a, (const __nv_bfloat16*)o, ldo, lse, (const __nv_bfloat16*)dO, lddo,
                                                    (__nv_bfloat16*)dq, lddq);
    attn::backward_dkv_kernel<16><<<bk, 256, 0, st>>>(a, (const __nv_bfloat16*)o, ldo, lse, (const __nv_bfloat16*)dO, lddo,
                                                     (__nv_bfloat16*)dk, lddk, (__nv_bfloat16*)dv, lddv);
  }
  return launched();
}

}  // extern "C"
