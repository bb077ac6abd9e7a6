/* Host-side co-serving scheduler arithmetic: the step-latency model, the SLO budget and the
 * fine-tuning admission of one step.  Everything here runs on the CPU; no entry point touches a
 * GPU.  It is the step BEFORE the mixed-batch layer (include/mlora.h): it decides how many
 * fine-tuning rows the next step's segment table carries.
 *
 *   Eq. I   (Section 4.1)  T = alpha * sum_i (n_i + B_d)^2 + beta * (T_in + B_d) + gamma * T_ft
 *                              + eps * K + c          for a step that holds prefill requests of
 *           lengths n_i (T_in = sum n_i), B_d decode requests, K cached key/value tokens and
 *           T_ft fine-tuning tokens whose activations are saved.
 *   Eq. II  (Section 4.1)  T = beta' * B_d + eps' * K + c'   for a decode-only step.
 *   Eq. III (Section 4.1)  budget = T_SLO - (t_now - t_arrival) of the earliest-arriving request.
 *   Algorithm 1 (Section 4.2)  admission of fine-tuning samples for one step, ending with the
 *           claim (buffer reserved, samples removed from the pool).
 *
 * Readings taken where the paper leaves a choice:
 *   - a fine-tuning sample joins the step as one more prefill entry (its length enters {n_i} and
 *     T_in) and its tokens also count in T_ft;
 *   - the inference-only batch is priced with the host's own mode (graph or eager coefficients),
 *     every batch that carries fine-tuning tokens with the eager coefficients;
 *   - the TTFT slack is +infinity for a batch without prefill requests, the TPOT slack is
 *     +infinity when no decode request exists (neither in the step nor deferred);
 *   - samples of equal length are taken in the order they entered the pool.
 * Times are in one unit of the caller's choice (the coefficients carry it); all are doubles.
 * Thread safety: a scheduler object must not be used from two threads at once. */
#ifndef MLORA_SCHED_H_
#define MLORA_SCHED_H_

#include <stdint.h>

#include "mlora.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct { double alpha, beta, gamma, eps, c; } mlora_mixed_coef_t;   /* Eq. I  */
typedef struct { double beta, eps, c; } mlora_decode_coef_t;                /* Eq. II */

/* Eq. I.  prefill_lens: host array of n_prefill lengths (fine-tuning samples included by the
 * caller, see the first reading above); may be NULL when n_prefill == 0.  Returns NaN on a NULL
 * coefficient pointer or a negative count. */
double mlora_predict_mixed(const mlora_mixed_coef_t* coef, const int32_t* prefill_lens, int32_t n_prefill,
                           int32_t n_decode, int64_t kv_tokens, int64_t ft_tokens);

/* Eq. II.  Returns NaN on a NULL coefficient pointer. */
double mlora_predict_decode(const mlora_decode_coef_t* coef, int32_t n_decode, int64_t kv_tokens);

/* Eq. III. */
double mlora_ttft_budget(double t_slo, double t_now, double t_arrival);

/* One observed step for the calibration fit: the batch composition and its measured time. */
typedef struct {
  const int32_t* prefill_lens;   /* host, n_prefill entries (may be NULL when n_prefill == 0) */
  int32_t n_prefill;
  int32_t n_decode;
  int64_t kv_tokens;
  int64_t ft_tokens;
  double seconds;                /* measured step time, in the caller's unit */
} mlora_observation_t;

/* Least-squares fit of Eq. I's coefficients to n_obs observations (Section 4.2, estimator
 * calibration).  fit_mask selects the coefficients that are fitted: bit 0 alpha, 1 beta, 2 gamma,
 * 3 eps, 4 c; the others are fixed at 0 (a workload without attention or a KV cache cannot
 * identify alpha and eps).  Solves the normal equations of the column-scaled system in long
 * double.  Errors: MLORA_ERR_INVALID_ARG (NULL, fit_mask 0 or > 31, fewer observations than
 * fitted coefficients), MLORA_ERR_UNSUPPORTED (the observations do not identify the chosen
 * coefficients: a singular system); *out is untouched on error. */
mlora_status_t mlora_fit_mixed(const mlora_observation_t* obs, int32_t n_obs, uint32_t fit_mask,
                               mlora_mixed_coef_t* out);

typedef struct {
  mlora_mixed_coef_t graph;      /* Eq. I for steps replayed from a captured graph            */
  mlora_mixed_coef_t eager;      /* Eq. I for eager steps (every step with fine-tuning rows)  */
  mlora_decode_coef_t decode;    /* Eq. II, prices the deferred decode batch                  */
  double t_slo_ttft;             /* TTFT SLO                                                  */
  double t_tpot;                 /* TPOT SLO                                                  */
  int64_t buffer_tokens;         /* capacity of the activation buffer in tokens (S_max at rest) */
  int32_t mixed_batch_host;      /* 1: the host forms prefill-decode mixed batches            */
  int32_t host_uses_graph;       /* 1: the inference-only step is priced with `graph`         */
} mlora_sched_config_t;

/* The inference batch the host is about to dispatch (B_inf) and the clock. */
typedef struct {
  const int32_t* prefill_lens;   /* host, n_prefill entries */
  int32_t n_prefill;
  int32_t n_decode;
  int64_t kv_tokens;
  double t_now;
  double earliest_arrival;       /* of the batch's prefill requests; ignored when n_prefill == 0 */
  int32_t wait_n_decode;         /* D_wait: decode requests deferred by this step (0: none)   */
  int64_t wait_kv_tokens;
} mlora_step_t;

typedef struct mlora_sched mlora_sched_t;

/* Creates a scheduler with an empty pool, an empty buffer and no backward running.
 * Errors: MLORA_ERR_INVALID_ARG (NULL, negative capacity). */
mlora_status_t mlora_sched_create(const mlora_sched_config_t* cfg, mlora_sched_t** out);
void mlora_sched_destroy(mlora_sched_t* s);

/* Replaces the coefficient sets (online refit, Section 4.2). */
mlora_status_t mlora_sched_set_coef(mlora_sched_t* s, const mlora_mixed_coef_t* graph,
                                    const mlora_mixed_coef_t* eager, const mlora_decode_coef_t* decode);

/* Online refinement (Section 4.2, estimator calibration: the estimator keeps refitting each execution
 * mode from the step times the host reports).  mlora_sched_observe stores one observed step
 * (composition as in mlora_observation_t, prefill_lens copied) in the ring of its mode - 0 eager,
 * 1 graph - which keeps the most recent `MLORA_SCHED_RING` (512) observations per mode.
 * mlora_sched_refit fits Eq. I to the ring of `mode` with mlora_fit_mixed(fit_mask) and, when the fit
 * succeeds, installs the result as that mode's coefficient set (coefficients outside fit_mask keep
 * their current values); *out (may be NULL) receives the installed set.  Errors: those of
 * mlora_fit_mixed (the set is left unchanged), MLORA_ERR_INVALID_ARG for a bad mode. */
#define MLORA_SCHED_RING 512
mlora_status_t mlora_sched_observe(mlora_sched_t* s, int32_t mode, const mlora_observation_t* obs);
int32_t mlora_sched_observations(const mlora_sched_t* s, int32_t mode);
mlora_status_t mlora_sched_refit(mlora_sched_t* s, int32_t mode, uint32_t fit_mask, mlora_mixed_coef_t* out);

/* Adds a fine-tuning sample of `tokens` (> 0) tokens to the pool Q_ft.  Ids are the caller's;
 * a duplicate id in the pool is MLORA_ERR_INVALID_ARG. */
mlora_status_t mlora_sched_pool_add(mlora_sched_t* s, int64_t sample_id, int32_t tokens);
int32_t mlora_sched_pool_size(const mlora_sched_t* s);
/* Remaining activation-buffer capacity S_max in tokens. */
int64_t mlora_sched_buffer_left(const mlora_sched_t* s);

/* The backward process state P_B: while it runs, admission returns nothing (Algorithm 1). */
mlora_status_t mlora_sched_set_backward_running(mlora_sched_t* s, int32_t running);

/* Algorithm 1 for one step, including the claim: the admitted samples leave the pool and their
 * tokens are reserved in the buffer.  out_ids (host, capacity `cap`) receives the sample ids in
 * admission order, out_tokens (may be NULL) their lengths, *n_out their number; at most `cap`
 * samples are admitted.  *budget (may be NULL) receives Delta, the step's latency budget (+inf
 * when unconstrained, NaN when admission was refused before it was computed).
 * Errors: MLORA_ERR_INVALID_ARG. */
mlora_status_t mlora_sched_admit(mlora_sched_t* s, const mlora_step_t* step, int64_t* out_ids,
                                 int32_t* out_tokens, int32_t cap, int32_t* n_out, double* budget);

/* Interrupted fine-tuning forward (Section 4.2): the samples return to the pool and their buffer
 * reservation is dropped.  tokens[i] must be what admission reported for ids[i]. */
mlora_status_t mlora_sched_requeue(mlora_sched_t* s, const int64_t* ids, const int32_t* tokens, int32_t n);

/* The backward consumed `tokens` tokens of saved activations: their buffer space is free again.
 * MLORA_ERR_INVALID_ARG when more is released than is reserved. */
mlora_status_t mlora_sched_buffer_release(mlora_sched_t* s, int64_t tokens);

#ifdef __cplusplus
}
#endif
#endif /* MLORA_SCHED_H_ */
