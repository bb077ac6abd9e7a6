/* The pieces of a Llama-3-style decoder layer around the multi-LoRA projections: RMSNorm, rotary
 * embedding, the SiLU gate and the residual add, forward and input gradient, bf16 on the device.
 * (Paper, Section 5: the model served and fine-tuned is Llama 3-8B; Section 3.2: by default only the
 * residual-stream input of each layer is saved per fine-tuning token and the backward recomputes the
 * layer from it, so these pieces run again there and their input gradients are needed.  The paper
 * describes no kernels for them; the base model is frozen, so no gradient of the norm gain exists.)
 * Attention is not part of this header.
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

/* out = a + b over n contiguous bf16 elements (n a multiple of 8); out may alias a or b. */
mlora_status_t mlora_add(const void* a, const void* b, void* out, int64_t n, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MLORA_LAYER_OPS_H_ */
