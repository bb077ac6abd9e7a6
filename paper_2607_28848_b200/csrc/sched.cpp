// Host-side scheduler arithmetic: Eq. I, II, III of Section 4.1 and Algorithm 1 of Section 4.2,
// plus the least-squares calibration of Eq. I.  No GPU code.
#include <algorithm>
#include <cmath>
#include <limits>
#include <new>
#include <vector>

#include "mlora_sched.h"

namespace {

struct PoolEntry {
  int64_t id;
  int32_t tokens;
  uint64_t seq;   // entry order; breaks ties between equal lengths
};

double mixed_cost(const mlora_mixed_coef_t& k, double attn, double t_in, int32_t n_decode, int64_t kv, int64_t ft) {
  return k.alpha * attn + k.beta * (t_in + (double)n_decode) + k.gamma * (double)ft + k.eps * (double)kv + k.c;
}

double attn_term(int32_t n, int32_t n_decode) {
  const double v = (double)n + (double)n_decode;
  return v * v;
}

}  // namespace

struct StoredObs {
  std::vector<int32_t> lens;
  int32_t n_decode;
  int64_t kv_tokens, ft_tokens;
  double seconds;
};

struct mlora_sched {
  mlora_sched_config_t cfg;
  std::vector<StoredObs> ring[2];       // observed steps per execution mode (0 eager, 1 graph)
  size_t ring_next[2] = {0, 0};
  std::vector<PoolEntry> pool;
  int64_t reserved = 0;
  uint64_t next_seq = 0;
  bool backward_running = false;
};

extern "C" {

double mlora_predict_mixed(const mlora_mixed_coef_t* coef, const int32_t* prefill_lens, int32_t n_prefill,
                           int32_t n_decode, int64_t kv_tokens, int64_t ft_tokens) {
  if (!coef || n_prefill < 0 || (n_prefill > 0 && !prefill_lens)) return std::numeric_limits<double>::quiet_NaN();
  double attn = 0.0, t_in = 0.0;
  for (int32_t i = 0; i < n_prefill; ++i) {
    attn += attn_term(prefill_lens[i], n_decode);
    t_in += (double)prefill_lens[i];
  }
  return mixed_cost(*coef, attn, t_in, n_decode, kv_tokens, ft_tokens);
}

double mlora_predict_decode(const mlora_decode_coef_t* coef, int32_t n_decode, int64_t kv_tokens) {
  if (!coef) return std::numeric_limits<double>::quiet_NaN();
  return coef->beta * (double)n_decode + coef->eps * (double)kv_tokens + coef->c;
}

double mlora_ttft_budget(double t_slo, double t_now, double t_arrival) { return t_slo - (t_now - t_arrival); }

mlora_status_t mlora_fit_mixed(const mlora_observation_t* obs, int32_t n_obs, uint32_t fit_mask,
                               mlora_mixed_coef_t* out) {
  if (!obs || !out || fit_mask == 0 || fit_mask > 31u || n_obs <= 0) return MLORA_ERR_INVALID_ARG;
  int cols[5], nc = 0;
  for (int j = 0; j < 5; ++j)
    if (fit_mask & (1u << j)) cols[nc++] = j;
  if (n_obs < nc) return MLORA_ERR_INVALID_ARG;
  std::vector<long double> X((size_t)n_obs * nc), y(n_obs);
  for (int32_t i = 0; i < n_obs; ++i) {
    const mlora_observation_t& o = obs[i];
    if (o.n_prefill < 0 || (o.n_prefill > 0 && !o.prefill_lens)) return MLORA_ERR_INVALID_ARG;
    long double f[5] = {0, 0, 0, 0, 1};
    for (int32_t p = 0; p < o.n_prefill; ++p) {
      f[0] += (long double)attn_term(o.prefill_lens[p], o.n_decode);
      f[1] += (long double)o.prefill_lens[p];
    }
    f[1] += (long double)o.n_decode;
    f[2] = (long double)o.ft_tokens;
    f[3] = (long double)o.kv_tokens;
    for (int j = 0; j < nc; ++j) X[(size_t)i * nc + j] = f[cols[j]];
    y[i] = (long double)o.seconds;
  }
  // column scaling keeps the normal equations' condition number in hand (tokens^2 beside 1)
  long double norm[5];
  for (int j = 0; j < nc; ++j) {
    long double s = 0;
    for (int32_t i = 0; i < n_obs; ++i) s += X[(size_t)i * nc + j] * X[(size_t)i * nc + j];
    if (!(s > 0)) return MLORA_ERR_UNSUPPORTED;
    norm[j] = sqrtl(s);
    for (int32_t i = 0; i < n_obs; ++i) X[(size_t)i * nc + j] /= norm[j];
  }
  long double G[5][6];
  for (int a = 0; a < nc; ++a) {
    for (int b = 0; b < nc; ++b) {
      long double s = 0;
      for (int32_t i = 0; i < n_obs; ++i) s += X[(size_t)i * nc + a] * X[(size_t)i * nc + b];
      G[a][b] = s;
    }
    long double s = 0;
    for (int32_t i = 0; i < n_obs; ++i) s += X[(size_t)i * nc + a] * y[i];
    G[a][nc] = s;
  }
  for (int p = 0; p < nc; ++p) {   // Gaussian elimination with partial pivoting
    int best = p;
    for (int r = p + 1; r < nc; ++r)
      if (fabsl(G[r][p]) > fabsl(G[best][p])) best = r;
    if (fabsl(G[best][p]) < 1e-13L) return MLORA_ERR_UNSUPPORTED;
    if (best != p)
      for (int c = 0; c <= nc; ++c) std::swap(G[p][c], G[best][c]);
    for (int r = p + 1; r < nc; ++r) {
      const long double m = G[r][p] / G[p][p];
      for (int c = p; c <= nc; ++c) G[r][c] -= m * G[p][c];
    }
  }
  long double sol[5];
  for (int p = nc - 1; p >= 0; --p) {
    long double s = G[p][nc];
    for (int c = p + 1; c < nc; ++c) s -= G[p][c] * sol[c];
    sol[p] = s / G[p][p];
  }
  double full[5] = {0, 0, 0, 0, 0};
  for (int j = 0; j < nc; ++j) full[cols[j]] = (double)(sol[j] / norm[j]);
  out->alpha = full[0]; out->beta = full[1]; out->gamma = full[2]; out->eps = full[3]; out->c = full[4];
  return MLORA_OK;
}

mlora_status_t mlora_sched_create(const mlora_sched_config_t* cfg, mlora_sched_t** out) {
  if (!cfg || !out || cfg->buffer_tokens < 0) return MLORA_ERR_INVALID_ARG;
  mlora_sched* s = new (std::nothrow) mlora_sched();
  if (!s) return MLORA_ERR_INVALID_ARG;
  s->cfg = *cfg;
  *out = s;
  return MLORA_OK;
}

void mlora_sched_destroy(mlora_sched_t* s) { delete s; }

mlora_status_t mlora_sched_set_coef(mlora_sched_t* s, const mlora_mixed_coef_t* graph,
                                    const mlora_mixed_coef_t* eager, const mlora_decode_coef_t* decode) {
  if (!s) return MLORA_ERR_INVALID_ARG;
  if (graph) s->cfg.graph = *graph;
  if (eager) s->cfg.eager = *eager;
  if (decode) s->cfg.decode = *decode;
  return MLORA_OK;
}

mlora_status_t mlora_sched_observe(mlora_sched_t* s, int32_t mode, const mlora_observation_t* obs) {
  if (!s || !obs || mode < 0 || mode > 1 || obs->n_prefill < 0 || (obs->n_prefill > 0 && !obs->prefill_lens))
    return MLORA_ERR_INVALID_ARG;
  StoredObs o;
  o.lens.assign(obs->prefill_lens, obs->prefill_lens + obs->n_prefill);
  o.n_decode = obs->n_decode; o.kv_tokens = obs->kv_tokens; o.ft_tokens = obs->ft_tokens; o.seconds = obs->seconds;
  std::vector<StoredObs>& r = s->ring[mode];
  if (r.size() < MLORA_SCHED_RING) {
    r.push_back(std::move(o));
  } else {
    r[s->ring_next[mode]] = std::move(o);
    s->ring_next[mode] = (s->ring_next[mode] + 1) % MLORA_SCHED_RING;
  }
  return MLORA_OK;
}

int32_t mlora_sched_observations(const mlora_sched_t* s, int32_t mode) {
  return (s && mode >= 0 && mode <= 1) ? (int32_t)s->ring[mode].size() : -1;
}

mlora_status_t mlora_sched_refit(mlora_sched_t* s, int32_t mode, uint32_t fit_mask, mlora_mixed_coef_t* out) {
  if (!s || mode < 0 || mode > 1) return MLORA_ERR_INVALID_ARG;
  const std::vector<StoredObs>& r = s->ring[mode];
  std::vector<mlora_observation_t> obs(r.size());
  for (size_t i = 0; i < r.size(); ++i)
    obs[i] = mlora_observation_t{r[i].lens.empty() ? nullptr : r[i].lens.data(), (int32_t)r[i].lens.size(), r[i].n_decode,
                                 r[i].kv_tokens, r[i].ft_tokens, r[i].seconds};
  mlora_mixed_coef_t fit;
  const mlora_status_t st = mlora_fit_mixed(obs.empty() ? nullptr : obs.data(), (int32_t)obs.size(), fit_mask, &fit);
  if (st != MLORA_OK) return st;
  mlora_mixed_coef_t& cur = mode == 1 ? s->cfg.graph : s->cfg.eager;
  if (fit_mask & 1u) cur.alpha = fit.alpha;
  if (fit_mask & 2u) cur.beta = fit.beta;
  if (fit_mask & 4u) cur.gamma = fit.gamma;
  if (fit_mask & 8u) cur.eps = fit.eps;
  if (fit_mask & 16u) cur.c = fit.c;
  if (out) *out = cur;
  return MLORA_OK;
}

mlora_status_t mlora_sched_pool_add(mlora_sched_t* s, int64_t sample_id, int32_t tokens) {
  if (!s || tokens <= 0) return MLORA_ERR_INVALID_ARG;
  for (const PoolEntry& e : s->pool)
    if (e.id == sample_id) return MLORA_ERR_INVALID_ARG;
  s->pool.push_back({sample_id, tokens, s->next_seq++});
  return MLORA_OK;
}

int32_t mlora_sched_pool_size(const mlora_sched_t* s) { return s ? (int32_t)s->pool.size() : -1; }

int64_t mlora_sched_buffer_left(const mlora_sched_t* s) { return s ? s->cfg.buffer_tokens - s->reserved : -1; }

mlora_status_t mlora_sched_set_backward_running(mlora_sched_t* s, int32_t running) {
  if (!s) return MLORA_ERR_INVALID_ARG;
  s->backward_running = running != 0;
  return MLORA_OK;
}

mlora_status_t mlora_sched_admit(mlora_sched_t* s, const mlora_step_t* step, int64_t* out_ids,
                                 int32_t* out_tokens, int32_t cap, int32_t* n_out, double* budget) {
  if (!s || !step || !n_out || cap < 0 || (cap > 0 && !out_ids) || step->n_prefill < 0 ||
      (step->n_prefill > 0 && !step->prefill_lens) || step->n_decode < 0 || step->wait_n_decode < 0)
    return MLORA_ERR_INVALID_ARG;
  *n_out = 0;
  if (budget) *budget = std::numeric_limits<double>::quiet_NaN();
  const int64_t s_max = s->cfg.buffer_tokens - s->reserved;
  if (s->backward_running || s_max <= 0 || s->pool.empty()) return MLORA_OK;
  const bool has_prefill = step->n_prefill > 0;
  if (!s->cfg.mixed_batch_host && !has_prefill) return MLORA_OK;

  const double inf = std::numeric_limits<double>::infinity();
  const double d_tt = has_prefill ? mlora_ttft_budget(s->cfg.t_slo_ttft, step->t_now, step->earliest_arrival) : inf;
  double d_tp = inf;
  if (step->n_decode > 0 || step->wait_n_decode > 0) {
    const double wait = step->wait_n_decode > 0
                            ? mlora_predict_decode(&s->cfg.decode, step->wait_n_decode, step->wait_kv_tokens)
                            : 0.0;
    d_tp = s->cfg.t_tpot - wait;
  }
  const double delta = std::min(d_tt, d_tp);
  if (budget) *budget = delta;

  double attn = 0.0, t_in = 0.0;
  for (int32_t i = 0; i < step->n_prefill; ++i) {
    attn += attn_term(step->prefill_lens[i], step->n_decode);
    t_in += (double)step->prefill_lens[i];
  }
  const mlora_mixed_coef_t& base = s->cfg.host_uses_graph ? s->cfg.graph : s->cfg.eager;
  if (mixed_cost(base, attn, t_in, step->n_decode, step->kv_tokens, 0) > delta) return MLORA_OK;

  std::vector<size_t> order(s->pool.size());
  for (size_t i = 0; i < order.size(); ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](size_t a, size_t b) {
    const PoolEntry &ea = s->pool[a], &eb = s->pool[b];
    return ea.tokens != eb.tokens ? ea.tokens < eb.tokens : ea.seq < eb.seq;
  });
  int64_t ft_tokens = 0;
  std::vector<char> taken(s->pool.size(), 0);
  int32_t n = 0;
  for (size_t oi = 0; oi < order.size() && n < cap; ++oi) {
    const PoolEntry& e = s->pool[order[oi]];
    const bool c1 = ft_tokens + e.tokens > s_max;
    const double attn2 = attn + attn_term(e.tokens, step->n_decode);
    const double t_in2 = t_in + (double)e.tokens;
    const bool c2 = mixed_cost(s->cfg.eager, attn2, t_in2, step->n_decode, step->kv_tokens, ft_tokens + e.tokens) > delta;
    if (c1 || c2) break;
    out_ids[n] = e.id;
    if (out_tokens) out_tokens[n] = e.tokens;
    ++n;
    taken[order[oi]] = 1;
    attn = attn2;
    t_in = t_in2;
    ft_tokens += e.tokens;
  }
  // the claim: reserve the buffer, remove the samples from the pool
  s->reserved += ft_tokens;
  size_t w = 0;
  for (size_t i = 0; i < s->pool.size(); ++i)
    if (!taken[i]) s->pool[w++] = s->pool[i];
  s->pool.resize(w);
  *n_out = n;
  return MLORA_OK;
}

mlora_status_t mlora_sched_requeue(mlora_sched_t* s, const int64_t* ids, const int32_t* tokens, int32_t n) {
  if (!s || n < 0 || (n > 0 && (!ids || !tokens))) return MLORA_ERR_INVALID_ARG;
  int64_t total = 0;
  for (int32_t i = 0; i < n; ++i) {
    if (tokens[i] <= 0) return MLORA_ERR_INVALID_ARG;
    total += tokens[i];
    for (const PoolEntry& e : s->pool)
      if (e.id == ids[i]) return MLORA_ERR_INVALID_ARG;
    for (int32_t j = 0; j < i; ++j)
      if (ids[j] == ids[i]) return MLORA_ERR_INVALID_ARG;
  }
  if (total > s->reserved) return MLORA_ERR_INVALID_ARG;
  s->reserved -= total;
  for (int32_t i = 0; i < n; ++i) s->pool.push_back({ids[i], tokens[i], s->next_seq++});
  return MLORA_OK;
}

mlora_status_t mlora_sched_buffer_release(mlora_sched_t* s, int64_t tokens) {
  if (!s || tokens < 0 || tokens > s->reserved) return MLORA_ERR_INVALID_ARG;
  s->reserved -= tokens;
  return MLORA_OK;
}

}  // extern "C"
