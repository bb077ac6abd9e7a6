/* The pieces of a Llama-3-style decoder layer around the multi-LoRA projections: RMSNorm, rotary
 * embedding, the SiLU gate and the residual add, forward and input gradient, bf16 on the device.
 * (Paper, Section 5: the model served and fine-tuned is Llama 3-8B; Section 3.2: by default only the
 * residual-stream input of each layer is saved per fine-tuning token and the backward recomputes the
 * layer from it, so these pieces run again there and their input gradients are needed.  The paper
 * describes no kernels for them; the base model is frozen, so no gradient of the norm gain exists.)
 * Attention is here too: for head size 128 three tcgen05 kernels (forward, dq, dk/dv: scores and
 * products in tensor memory, operands by TMA, every wait bounded with its status read by
 * mlora_layer_ops_poll_status), for head size 64 plain CUDA-core kernels (one warp per row and head).
 *
 * All pointers are device pointers on the current device, all buffers borrowed; leading dimensions
 * (ld*) are in elements; rows and element counts must keep 16-byte alignment as stated per call.
 * Calls are asynchronous on `cuda_stream`, allocate nothing, never synchronise.
 * Errors: MLORA_ERR_INVALID_ARG (null pointer, negative size), MLORA_ERR_UNSUPPORTED (alignment /
 * divisibility), MLORA_ERR_CUDA (launch failed). */
#ifndef MLORA_LAYER_OPS_H_
#define MLORA_LAYER_OPS_H_

#include <stdint.h>

#include "mlora.h"

#ifdef __cplusplus
extern "C" {
#endif

/* y[t, :] = x[t, :] * rsqrt(mean_k x[t, k]^2 + eps) * gain.  x, y bf16 [n_rows, d] (ldx, ldy >= d,
 * multiples of 8), gain fp32 [d]; d a multiple of 8. */
mlora_status_t mlora_rmsnorm_forward(const void* x, int64_t ldx, const float* gain, void* y, int64_t ldy,
                                     int32_t n_rows, int32_t d, float eps, void* cuda_stream);

/* dx = rstd * (u - xh * mean(u * xh)) with u = gain * dy, xh = x * rstd, rstd recomputed from x. */
mlora_status_t mlora_rmsnorm_backward(const void* x, int64_t ldx, const float* gain, const void* dy, int64_t lddy,
                                      void* dx, int64_t lddx, int32_t n_rows, int32_t d, float eps, void* cuda_stream);

/* Rotary embedding of x bf16 [n_rows, n_heads, d_head] (row stride ldx): elements i and i + d_head/2
 * of every head are rotated by the angle pos[t] * theta^(-2 i / d_head) (reading: the "rotate half"
 * pairing of the Llama code base).  transpose != 0 applies the transposed rotation, which is the
 * input gradient of the forward.  y may alias x.  pos int32 [n_rows]; d_head a multiple of 16. */
mlora_status_t mlora_rope(const void* x, int64_t ldx, void* y, int64_t ldy, const int32_t* pos, int32_t n_rows,
                          int32_t n_heads, int32_t d_head, float theta, int32_t transpose, void* cuda_stream);

/* m = silu(g) * u, element-wise over n elements (contiguous bf16 buffers, n a multiple of 8). */
mlora_status_t mlora_swiglu_forward(const void* g, const void* u, void* m, int64_t n, void* cuda_stream);

/* dg = dm * u * s * (1 + g * (1 - s)), du = dm * g * s with s = 1 / (1 + exp(-g)). */
mlora_status_t mlora_swiglu_backward(const void* g, const void* u, const void* dm, void* dg, void* du, int64_t n,
                                     void* cuda_stream);

/* out = a + b over n contiguous bf16 elements (n a multiple of 8); out may alias a or b.  The residual
 * connections of the forward, and in the backward the sum of the gradients of a tensor that feeds several
 * consumers (layer input -> norm and residual, normed input -> q, k and v or gate and up). */
mlora_status_t mlora_add(const void* a, const void* b, void* out, int64_t n, void* cuda_stream);

/* Causal softmax attention inside each sequence of a packed batch, grouped-query heads:
 *   o[i, h] = sum_{j <= i, same sequence} softmax_j(q[i, h] . k[j, h / (n_heads / n_kv)] / sqrt(d_head)) v[j, ...]
 * q, o bf16 [n_rows, n_heads * d_head] (row strides ldq, ldo), k, v bf16 [n_rows, n_kv * d_head];
 * seq_start[i] = first row of row i's sequence, seq_end[i] = one past its last row (int32 [n_rows]; the
 * rows of a sequence are consecutive); lse fp32 [n_rows, n_heads] receives log(sum_j exp(s_ij)), which the
 * backward needs.  d_head is 64 or 128 (128: tcgen05 tensor-core kernel, 64: CUDA cores); n_heads a multiple
 * of n_kv; seq_start must not decrease from row to row (sequences are stored one after the other). */
mlora_status_t mlora_attention_forward(const void* q, int64_t ldq, const void* k, int64_t ldk, const void* v, int64_t ldv,
                                       void* o, int64_t ldo, float* lse, const int32_t* seq_start, const int32_t* seq_end,
                                       int32_t n_rows, int32_t n_heads, int32_t n_kv, int32_t d_head, void* cuda_stream);

/* The forward for d_head = 128 runs on the tensor cores with bounded waits inside the kernel; a wait
 * that runs out makes the kernel return early and leaves MLORA_ERR_DEVICE_TIMEOUT in a device status
 * word.  This call synchronises the stream, returns that word (MLORA_OK when nothing happened) and
 * clears it.  The outputs of a call that timed out are undefined. */
mlora_status_t mlora_layer_ops_poll_status(void* cuda_stream);

/* Gradients of the above for a given dO: dq like q, dk and dv like k and v (each element written once; the
 * sums over the query heads that share a kv head are inside).  o and lse are the forward's outputs.
 * d_head = 128 runs on the tensor cores like the forward (the probabilities, recomputed from lse, and dS
 * enter the products rounded to bf16; accumulation is fp32); d_head = 64 on the CUDA cores in fp32. */
mlora_status_t mlora_attention_backward(const void* q, int64_t ldq, const void* k, int64_t ldk, const void* v, int64_t ldv,
                                        const void* o, int64_t ldo, const float* lse, const void* dO, int64_t lddo,
                                        void* dq, int64_t lddq, void* dk, int64_t lddk, void* dv, int64_t lddv,
                                        const int32_t* seq_start, const int32_t* seq_end, int32_t n_rows,
                                        int32_t n_heads, int32_t n_kv, int32_t d_head, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MLORA_LAYER_OPS_H_ */
