/*
 * mlora.h - C ABI of the mixed-batch multi-LoRA linear layer for NVIDIA B200 (sm_100a).
 *
 * One call runs inference rows (prefill and decode tokens) and LoRA fine-tuning rows
 * through ONE pass over a frozen base weight, every row applying the low-rank adapter it
 * is bound to; fine-tuning rows additionally leave behind the activations their backward
 * needs.  A second call computes the LoRA gradients (and the input gradient) for those rows.
 *
 * Row-vector convention.  For a row x bound to adapter a:
 *        y = x W + s_a (x A_a^T) B_a
 * with W [d_in, d_out], A_a [rank, d_in], B_a [rank, d_out], s_a = alpha_a / rank.
 * (Paper, Section 2.2: frozen W plus a trainable rank-r product, W_eff = W + B A; its A is
 * A_a, its B is B_a transposed.  The scaling s comes from Section 5, "Fine-tuning
 * Workload": r = 16, alpha = 32.)
 *
 * General rules
 *  - Every pointer named "device" is a CUDA device pointer on the context's device; every
 *    other pointer is a host pointer.  All device buffers are BORROWED: the library never
 *    frees them and does not touch them after the work queued on the stream has finished.
 *  - Matrices are row-major; leading dimensions (ld*) are in ELEMENTS.
 *  - Calls return an mlora_status_t.  Argument errors are found on the host before
 *    anything is launched.  mlora_mixed_forward / mlora_backward are asynchronous on the
 *    given stream, allocate nothing and never synchronise.
 *  - There is no CPU fallback: without an sm_100 device mlora_create fails with
 *    MLORA_ERR_ARCH and no compute entry point can be used.
 *  - A context owns workspaces (the rank-r intermediate of the running call, the GEMM's low-rank
 *    operand, partial sums) that serve ONE compute call at a time: the calls on a context must be
 *    queued on one stream, or on streams ordered after one another.  A context is used from one
 *    host thread at a time; different contexts (one per GPU, or several on one) are independent.
 *  - The library never aborts the process and throws nothing across this boundary.
 */
#ifndef MLORA_H_
#define MLORA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mlora_ctx mlora_ctx;     /* per-device state: workspace, status word        */
typedef struct mlora_plan mlora_plan;   /* a validated segment table and its device tables */

/* One contiguous run of rows bound to one adapter (paper, Section 2.2 "multi-LoRA batching":
 * adapter-bound requests share one base pass; Section 3.2 "Mixed forward batch": a
 * fine-tuning sample is one more prefill-like entry routed to its adapter).
 * adapter_id = -1 means "base weight only"; is_finetune != 0 marks rows whose activations
 * are saved and which take part in the backward. */
typedef struct {
  int32_t row_start;
  int32_t row_len;
  int32_t adapter_id;
  int32_t is_finetune;
} mlora_segment_t;

typedef enum { MLORA_F32 = 0, MLORA_BF16 = 1 } mlora_dtype_t;

typedef enum {
  MLORA_OK = 0,
  MLORA_ERR_INVALID_ARG = 1,     /* null pointer, negative size, bad enum                       */
  MLORA_ERR_SEGMENT_RANGE = 2,   /* a segment leaves [0, n_rows) or has negative length         */
  MLORA_ERR_SEGMENT_OVERLAP = 3, /* two segments share a row                                    */
  MLORA_ERR_ADAPTER_ID = 4,      /* adapter id outside [-1, n_adapters), or fine-tune with -1   */
  MLORA_ERR_SAVE_CAPACITY = 5,   /* fine-tune rows do not fit the activation buffer             */
  MLORA_ERR_UNSUPPORTED = 6,     /* shape / rank / alignment outside what the kernels handle    */
  MLORA_ERR_ARCH = 7,            /* no CUDA device of compute capability 10.x                   */
  MLORA_ERR_CUDA = 8,            /* a CUDA runtime or driver call failed                        */
  MLORA_ERR_DEVICE_TIMEOUT = 9,  /* a bounded wait inside a kernel ran out (see poll_status)    */
  MLORA_CANCELLED = 10           /* the caller's cancel flag was raised; the call stopped early */
} mlora_status_t;

/* One projection.  dtype is the storage type of X, W, A, B, Y, dY, dX and x_save.
 *   MLORA_BF16: tensor-core path; needs d_in, d_out multiples of 64, rank in {8,16,32,64,128},
 *               ldw a multiple of 8 and every base pointer 16-byte aligned.
 *   MLORA_F32 : plain fp32 path (small layers, correctness work); rank <= 128. */
typedef struct {
  int32_t d_in, d_out, rank, n_adapters;
  int32_t dtype;          /* mlora_dtype_t */
  const void* W;          /* device [d_in, d_out], row stride ldw; frozen                    */
  int64_t ldw;
  const void* A_all;      /* device [n_adapters, rank, d_in], dense                           */
  const void* B_all;      /* device [n_adapters, rank, d_out], dense                          */
  const float* scale;     /* device [n_adapters] fp32, s_a = alpha_a / rank                   */
} mlora_layer_t;

/* ---- context ---------------------------------------------------------------------------*/

/* Creates the per-device state on CUDA device `device`, including two workspaces of fixed size
 * that are allocated here so that no compute call allocates: 64 MiB for the fp32 partial products
 * of K-split GEMMs and SMs x 128 KiB for the partial sums of row-split gradient groups.  Fails
 * with MLORA_ERR_ARCH when the device is not compute capability 10.x, MLORA_ERR_CUDA when the
 * runtime cannot be used or the workspaces cannot be allocated. */
mlora_status_t mlora_create(mlora_ctx** ctx, int device);
void mlora_destroy(mlora_ctx* ctx);

/* ---- plan: segment table -> validated routing ------------------------------------------*/

/* Validates `segs` (host array of n_segs entries) for a batch of n_rows rows and n_adapters
 * adapters, and derives: the adapter of every row, the save offset of every fine-tuning
 * segment (exclusive prefix sum of the fine-tuning lengths in TABLE ORDER; paper, Section
 * 3.2: captured activations are appended to a buffer the backward consumes), the gradient
 * slots (one per distinct fine-tuning adapter, in order of first appearance) and the tile
 * schedules of the kernels.  Segments may come in any order; zero-length segments are legal;
 * rows covered by no segment use the base weight only.
 * With ctx == NULL the plan is host-only (for inspection; it cannot be executed).  With a
 * context the tables are uploaded (through a buffer pair - device tables and pinned staging - taken
 * from a pool inside the context, on the default stream, and the upload is waited for) and the
 * context's workspaces are enlarged if this batch is larger than any before.  mlora_plan_destroy
 * waits for the device and gives the pair back to the pool, so in steady state the two calls make no
 * cudaMalloc / cudaMallocHost / cudaFree (0.14 ms for a table of a thousand segments; each of those
 * calls costs milliseconds when the driver has to map or unmap pages).  They still synchronise: a
 * plan that lives for one step is what mlora_plan_create_async below is for.  The compute calls never
 * allocate or synchronise.  An enlarged workspace is a NEW block; the block it replaces stays allocated until
 * mlora_destroy, so kernels already queued and CUDA graphs captured earlier keep working on memory
 * that is still theirs - creating a larger plan never invalidates an earlier plan or graph.
 * Errors: MLORA_ERR_SEGMENT_RANGE, MLORA_ERR_SEGMENT_OVERLAP, MLORA_ERR_ADAPTER_ID,
 * MLORA_ERR_INVALID_ARG, MLORA_ERR_CUDA. */
mlora_status_t mlora_plan_create(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs,
                                 int32_t n_rows, int32_t n_adapters, mlora_plan** plan);
/* The same plan for adapters that have ranks of their own (Section 2.2: a serving system hosts many
 * adapters over one frozen base model; nothing makes them share a rank).  adapter_rank: HOST array [n_adapters], 1 <= r_a <= 128; NULL makes
 * this call mlora_plan_create.  Storage does not change: every adapter still occupies `rank` rows of
 * A_all and B_all in each layer, rows r_a .. rank - 1 zero, and gradients come back in that shape with
 * those rows zero.  What changes is the work: in the base product's fused expand a group of rows is
 * as wide as its adapter's rank rounded up to 16, not as wide as the layer's padded rank, so the
 * extra K-blocks of a 256-row tile number ceil(sum of those widths / 64) instead of
 * ceil(groups * rank / 64); and the tcgen05 shrink (layer ranks 64 and 128) reads, per block of rows,
 * only the first 16 / 32 / 64 / 128 rows of the adapter's matrices that its rank needs, and the
 * tcgen05 gradient kernel contracts only those rows of a slot's gradient (the rest is written as
 * zero).  (The mma.sync kernels of the lower layer ranks still run over all `rank` rows.)
 * A plan made this way serves layers with rank % 16 == 0 and rank >= every r_a; other layers are
 * refused by the compute calls with MLORA_ERR_INVALID_ARG.  Errors as mlora_plan_create, plus
 * MLORA_ERR_INVALID_ARG for a rank outside [1, 128]. */
mlora_status_t mlora_plan_create_ranked(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs,
                                        int32_t n_rows, int32_t n_adapters, const int32_t* adapter_rank,
                                        mlora_plan** plan);
void mlora_plan_destroy(mlora_plan* plan);

/* Stream-ordered variant for serving loops, where every step has a new batch mix (paper,
 * Section 4.2: the admission decision is taken per scheduling step): the tables go into a buffer
 * pair (device + pinned host staging) taken from a pool inside the context and are uploaded with
 * an asynchronous copy on `cuda_stream`; compute calls that use the plan must be queued on that
 * same stream (or on one ordered after it).  In steady state the call neither allocates nor
 * synchronises (a pool miss allocates a pair, a batch larger than any before grows the context's
 * workspace as mlora_plan_create does - neither inside a stream capture).  ctx must not be NULL.
 * mlora_plan_release gives the pair back: it records an event on `cuda_stream` (the stream the
 * plan's last compute call was queued on) and the pair is reused once that event has passed; the
 * plan handle is invalid afterwards.  mlora_plan_destroy also accepts such a plan (it frees the
 * pair, waiting for the device).  Errors: as mlora_plan_create. */
mlora_status_t mlora_plan_create_async(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs,
                                       int32_t n_rows, int32_t n_adapters, void* cuda_stream,
                                       mlora_plan** plan);
/* mlora_plan_create_async for adapters with ranks of their own (see mlora_plan_create_ranked). */
mlora_status_t mlora_plan_create_ranked_async(mlora_ctx* ctx, const mlora_segment_t* segs, int32_t n_segs,
                                              int32_t n_rows, int32_t n_adapters, const int32_t* adapter_rank,
                                              void* cuda_stream, mlora_plan** plan);
mlora_status_t mlora_plan_release(mlora_plan* plan, void* cuda_stream);

int32_t mlora_plan_rows(const mlora_plan* plan);        /* n_rows                              */
int32_t mlora_plan_ft_rows(const mlora_plan* plan);     /* total fine-tuning rows, T_ft        */
/* Writes up to `cap` adapter ids, slot g -> adapter id, and returns the number of slots. */
int32_t mlora_plan_ft_adapters(const mlora_plan* plan, int32_t* ids, int32_t cap);
/* Inspection: out[k] = save offset of segment k, or -1 when it is not a fine-tuning segment
 * (n_segs entries); row_adapter[t] = adapter of row t or -1 (n_rows entries). Either may be NULL. */
mlora_status_t mlora_plan_describe(const mlora_plan* plan, int32_t* seg_save_offset, int32_t* row_adapter);
/* Cost view of the fused expand: for every 256-row tile of the batch, how many columns its low-rank
 * operand has = the contraction depth the tile adds to the base product (in steps of 64 it is the
 * tile's count of extra K-blocks).  Without per-adapter ranks that is (distinct adapters in the
 * tile) * rank; a plan made by mlora_plan_create_ranked counts each adapter with its own rank
 * rounded up to 16, and `rank` is ignored.  Writes up to cap entries into cols and returns the number
 * of tiles, ceil(n_rows / 256).  Works without a context (host-only plans). */
int32_t mlora_plan_lowrank_columns(const mlora_plan* plan, int32_t rank, int32_t* cols, int32_t cap);

/* ---- forward ---------------------------------------------------------------------------*/

/* Y[t,:] = X[t,:] W + s_a (X[t,:] A_a^T) B_a for every row t (a = adapter of t; base only when
 * a = -1), inference and fine-tuning rows in the same pass (paper, Section 2.2 multi-LoRA
 * batching; Section 3.2 "Mixed forward batch").  For fine-tuning rows only, the row of X and the
 * UNSCALED rank-r product u = x A_a^T are written to the caller's activation buffer at row
 *        save_row_base + save_offset(segment) + i          (i = row index inside the segment)
 * (paper, Section 3.2: activation capture for fine-tuning rows; intermediates may be cached to
 * avoid recomputation).  Inference rows save nothing.
 *   X       device [n_rows, d_in], row stride ldx          (read)
 *   Y       device [n_rows, d_out], row stride ldy         (written once, every row)
 *   x_save  device [save_capacity_rows, d_in] dense, layer dtype; NULL skips the copy of X
 *   u_save  device [save_capacity_rows, rank] dense fp32; required when the plan has
 *           fine-tuning rows
 * save_row_base + T_ft > save_capacity_rows -> MLORA_ERR_SAVE_CAPACITY (nothing launched).
 * Other errors: MLORA_ERR_INVALID_ARG, MLORA_ERR_ADAPTER_ID (plan built for more adapters than
 * the layer has), MLORA_ERR_UNSUPPORTED, MLORA_ERR_CUDA. */
mlora_status_t mlora_mixed_forward(mlora_ctx* ctx, const mlora_layer_t* layer, const mlora_plan* plan,
                                   const void* X, int64_t ldx, void* Y, int64_t ldy,
                                   void* x_save, float* u_save,
                                   int64_t save_row_base, int64_t save_capacity_rows,
                                   void* cuda_stream);

/* ---- backward --------------------------------------------------------------------------*/

/* LoRA backward for the plan's fine-tuning rows (paper, Section 3.2 "Backward subprocess":
 * LoRA gradients are computed from the saved activations; the formulas are the chain rule of
 * the forward).  All row-indexed buffers are in SAVE ORDER: row m is the m-th fine-tuning row
 * (the pointers address the first row this plan saved, i.e. the caller adds save_row_base).
 *        V    = s_a dY B_a^T                           [T_ft, rank]  (internal)
 *        dB_g (+)= sum over rows of slot g  s_a u^T dY [rank, d_out]
 *        dA_g (+)= sum over rows of slot g  V^T x      [rank, d_in]
 *        dX   = dY W^T + V A_a                         [T_ft, d_in]
 *   dY_ft   device [T_ft, d_out], row stride lddy, layer dtype      (read)
 *   x_save  device [T_ft, d_in] dense, layer dtype                  (read)
 *   u_save  device [T_ft, rank] dense fp32                          (read)
 *   dA      device [n_slots, rank, d_in]  fp32, dense (same orientation as A_all)
 *   dB      device [n_slots, rank, d_out] fp32, dense (same orientation as B_all)
 *   dX_ft   device [T_ft, d_in], row stride lddx, layer dtype; NULL skips dX
 *   accumulate  0: dA, dB are overwritten;  nonzero: the new gradients are added to them
 * Slot g belongs to adapter mlora_plan_ft_adapters()[g]; several fine-tuning segments on one
 * adapter add into one slot.  A plan without fine-tuning rows makes this a no-op. */
mlora_status_t mlora_backward(mlora_ctx* ctx, const mlora_layer_t* layer, const mlora_plan* plan,
                              const void* dY_ft, int64_t lddy,
                              const void* x_save, const float* u_save,
                              float* dA, float* dB, void* dX_ft, int64_t lddx,
                              int32_t accumulate, void* cuda_stream);

/* ---- cooperative cancellation --------------------------------------------------------------*/

/* Registers a HOST flag (for example a word in pinned or ordinary host memory that another
 * thread writes) that mlora_mixed_forward, mlora_backward and mlora_adamw_update read before each
 * kernel they launch; NULL unregisters.  When it is non-zero the call launches nothing further and
 * returns MLORA_CANCELLED.  Kernels already queued still run to completion, so the GPU is free
 * within one kernel's time; the outputs of the interrupted call are incomplete and the caller
 * drops them (for a forward: do not advance save_row_base, so the partial activations are
 * overwritten by the next step; the interrupted rows go back to the caller's pool).
 * (Paper, Section 4 "Backward preemption" and "Fine-tuning forward interruption": a grant flag /
 * abort signal polled at layer boundaries, discarding partial activations.  Here the boundary is
 * finer - between the two to four kernels of one projection - and the flag is read on the host,
 * which learns of the request before its next launch, so no kernel ever waits on it.) */
mlora_status_t mlora_set_cancel_flag(mlora_ctx* ctx, const volatile int32_t* host_flag);

/* ---- LoRA dropout on the fine-tuning rows --------------------------------------------------*/

/* Switches dropout of the low-rank branch's input on (0 < p < 1) or off (p == 0) for the compute
 * calls that follow on this context.  (Paper, Section 5 "Fine-tuning Workload": the adapter is
 * trained with dropout 0.05; reading: the usual LoRA placement y = x W + s B A dropout(x), on
 * fine-tuning rows only - inference rows and the base product never see it.)
 * The keep decision of element (m, k) - m the row's place in the batch's save order, counted from
 * the first row the plan saves, k the input column - is output number c + 1 of the SplitMix64
 * stream started at `seed`, c = m * 2^32 + (k >> 2); its 16-bit field k & 3 is compared with
 * round(p * 65536) (ties to even), values below it are dropped; kept elements count 1 / (1 - p).
 * Forward:  u_save and Y use the dropped input, x_save keeps the row as it is.
 * Backward: dA = (V / (1 - p))^T (x_save * keep), dX = dY W^T + (V A) * keep / (1 - p); V and dB
 * keep their form.  The forward and the backward of one batch must run under the same (p, seed);
 * the caller changes the seed from step to step and from layer to layer.  A captured graph keeps
 * the values it was captured with.
 * Supported for fp32 layers and for bf16 layers of every rank on the default kernel path (the
 * mma.sync kernels mask the rows as they read them: the streaming kernels up to rank 64, the
 * per-item kernels at rank 128); under kernel variant 2 only at rank 128, otherwise the compute
 * call returns MLORA_ERR_UNSUPPORTED.  With dropout on, the low-rank part of dX is added by one
 * extra elementwise kernel after the base product.
 * Errors: MLORA_ERR_INVALID_ARG (NULL context, p outside [0, 1)). */
mlora_status_t mlora_set_dropout(mlora_ctx* ctx, double p, uint64_t seed);

/* ---- optimizer step on the fine-tuned adapters ------------------------------------------*/

/* AdamW hyper-parameters (paper, Section 5 "Fine-tuning Workload": AdamW, learning rate 1e-3,
 * weight decay 0.01; betas and epsilon are not stated there, the usual 0.9 / 0.999 / 1e-8 are the
 * documented defaults).  `step` is the 1-based index of this update (bias correction). */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int32_t step;
} mlora_adamw_t;

/* Applies one decoupled-weight-decay Adam update to the adapters the plan fine-tunes, consuming
 * the gradients mlora_backward produced, and rewrites those adapters' rows of A_all and B_all in
 * place (paper, Section 3.2 "Backward subprocess": optimizer updates are applied directly to the
 * shared adapter weights):
 *        w <- w - lr wd w;  m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
 *        w <- w - lr (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps)
 * All arithmetic is fp32 on fp32 master weights; the layer's stored weights (layer dtype) are the
 * master weights rounded to nearest even.  One fused, vectorised pass over 30 bytes per element.
 *   layer     A_all / B_all are WRITTEN for the plan's fine-tuning adapters (only those rows)
 *   dA, dB    device fp32 [n_slots, rank, d_in] / [n_slots, rank, d_out]   (read)
 *   wA, wB    device fp32 master weights, same shapes, slot-indexed        (read + written)
 *   mA, vA, mB, vB  device fp32 first / second moments, same shapes        (read + written)
 * Slot g belongs to adapter mlora_plan_ft_adapters()[g].  The caller initialises the master
 * weights from the adapters once and zeroes the moments.  A plan without fine-tuning rows makes
 * this a no-op.  Errors: MLORA_ERR_INVALID_ARG (null pointers, step < 1, betas outside [0,1)),
 * MLORA_ERR_ADAPTER_ID, MLORA_ERR_CUDA.  Asynchronous on the stream; allocates nothing. */
mlora_status_t mlora_adamw_update(mlora_ctx* ctx, const mlora_layer_t* layer, const mlora_plan* plan,
                                  const float* dA, const float* dB, float* wA, float* wB,
                                  float* mA, float* vA, float* mB, float* vB,
                                  const mlora_adamw_t* hp, void* cuda_stream);

/* ---- status / diagnostics --------------------------------------------------------------*/

/* Synchronises the stream and returns the device status word: MLORA_OK, or
 * MLORA_ERR_DEVICE_TIMEOUT when a bounded wait inside a kernel gave up (the kernel then
 * released its resources and returned; its outputs are invalid).  Clears the word, and after a
 * timeout also the arrival counters of work items that several CTAs share (a kernel that gave up may
 * have left them partly counted), so that the next compute call starts from a clean state. */
mlora_status_t mlora_poll_status(mlora_ctx* ctx, void* cuda_stream);
const char* mlora_status_string(mlora_status_t s);

/* Self-test of that report path (the paper has no counterpart; it belongs to this library's rule that no
 * wait inside a kernel is unbounded).  Queues one tiny kernel whose only work is to wait, with the wait
 * helper of the streaming kernels, on a barrier that nothing ever arrives at, for `polls` polls
 * (1 .. 2^20; a thousand take microseconds).  The wait runs out, the kernel records
 * MLORA_ERR_DEVICE_TIMEOUT in the status word and returns normally: nothing faults or hangs and the
 * context stays usable.  The next mlora_poll_status therefore returns MLORA_ERR_DEVICE_TIMEOUT, clears the
 * word together with the arrival counters of split work items, and the poll after that returns MLORA_OK.
 * Errors: MLORA_ERR_INVALID_ARG (NULL context, polls out of range), MLORA_ERR_CUDA. */
mlora_status_t mlora_selftest_timeout(mlora_ctx* ctx, uint32_t polls, void* cuda_stream);

/* Number of kernels the library has launched on this context since it was created. */
int64_t mlora_launch_count(const mlora_ctx* ctx);

/* Per-kernel timing.  mlora_profile_enable(ctx, n) with n > 0 creates n CUDA event pairs (this
 * allocates; call it outside any timed or captured region) and makes every later kernel launch
 * of this context record one pair around itself on the launching stream, until the pairs run
 * out; n = 0 switches recording off and frees the events.  mlora_profile_collect synchronises
 * the device, writes for each recorded launch its kind (0 shrink, 1 forward GEMM, 2 input-gradient
 * GEMM, 3 gradient kernel, 4 CUDA-core kernels, 5 optimizer update, 6 reduction kernel of a K-split GEMM) and its
 * duration in milliseconds into the host
 * arrays (up to cap entries), forgets the records and returns how many there were. */
mlora_status_t mlora_profile_enable(mlora_ctx* ctx, int32_t max_records);
int32_t mlora_profile_collect(mlora_ctx* ctx, int32_t* kinds, float* ms, int32_t cap);

/* Selects kernel variants for MLORA_BF16 layers: 0 = defaults (two-SM tcgen05 tensor-core GEMM; rank <= 16:
 * streaming mma.sync shrink and gradient kernels; rank 32, 64 and 128: the tcgen05 shrink with its finish
 * kernel for U = X A^T and V = s dY B^T wherever the rows come in runs of eight (rank 128: four) or more
 * per adapter on average, and the tcgen05 gradient kernel); 1 = the plain CUDA-core kernels for every step (a slow
 * cross-check used by the tests); 2 = defaults, but the per-item mma.sync shrink and gradient kernels
 * for every rank; 3 = defaults, but the one-SM tensor-core GEMM;
 * 4 = defaults, but the two-SM GEMM never splits K (by default a product with too few output
 * tiles for the SMs is cut into K slices whose fp32 partials a small kernel adds up);
 * 5 = defaults, but both gradients on the mma.sync kernels for every rank;
 * 6 = defaults, but every rank-r product on the tcgen05 kernels for every rank: U, V and both gradients
 * (with dropout on, everything stays on the mma.sync kernels);
 * 7 = defaults, but the two-SM GEMM always deals its tiles out round robin (by default a batch whose
 * 256-row tiles differ much in their number of adapter groups gets, per shape it is used with, a list
 * that spreads the tiles over the CTA pairs by cost; the list is built on the host at the first such
 * call, kept with the plan, and never built while the stream is being captured). */
mlora_status_t mlora_set_gemm_path(mlora_ctx* ctx, int32_t path);

/* ---- forward without any allocation -----------------------------------------------------*/

/* (The paper has no counterpart for this entry point; it exists for integration reasons.)
 *
 * Some callers are not allowed to allocate device memory at all: an inference engine that hands
 * its whole memory budget to its own pool at start-up and treats any later cudaMalloc as a bug,
 * a worker that attaches to another process's buffers and owns no memory of its own, or code
 * running where an allocation would stall the device (cudaMalloc synchronises).  The regular
 * path needs a context and a plan, and both allocate.  This call needs neither: it computes
 *        Y[t,:] = X[t,:] W + s_a (X[t,:] A_a^T) B_a,    a = row_adapter[t]  (-1: base only)
 * for a small batch of inference rows with the plain CUDA-core kernels, keeping the rank-r
 * intermediate x A_a^T in a fixed scratch array that is part of the library image
 * (MLORA_NOALLOC_MAX_ROWS x 128 floats = 256 KiB, held by every GPU that loads the library until
 * the process exits).  It calls no cudaMalloc, cudaFree or allocating library routine.
 *   layer        as for mlora_mixed_forward (either dtype; no 64-multiple requirement here)
 *   row_adapter  device [n_rows] int32, each in [-1, layer->n_adapters).  The table lives on the device, so
 *                the host cannot check it; the kernels treat an id outside that range as -1 (the row
 *                gets the base product only) and never index the adapter tables with it
 *   X, Y         device [n_rows, d_in] / [n_rows, d_out], row strides ldx / ldy
 * Runs on the CURRENT device, asynchronously on the given stream.  Nothing is saved for
 * fine-tuning; use the planned path for that.
 * Limits and errors: n_rows > MLORA_NOALLOC_MAX_ROWS or rank > 128 -> MLORA_ERR_UNSUPPORTED
 * (nothing launched); null pointers / bad sizes -> MLORA_ERR_INVALID_ARG; CUDA failures ->
 * MLORA_ERR_CUDA.  n_rows = 0 is a no-op.
 * First call on a device: it looks up the scratch array's device address (no allocation, but a
 * runtime query), so make that first call before starting any stream capture.
 * Sharing: every call on a device uses the same scratch and leaves its contents behind.  Each call
 * rewrites all entries it later reads, so nothing needs clearing between calls; but two calls
 * whose work overlaps on the GPU (different streams, no ordering) race on it - serialise them. */
#define MLORA_NOALLOC_MAX_ROWS 512
mlora_status_t mlora_forward_noalloc(const mlora_layer_t* layer, const int32_t* row_adapter, int32_t n_rows,
                                     const void* X, int64_t ldx, void* Y, int64_t ldy, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MLORA_H_ */
