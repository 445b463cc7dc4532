// C ABI of libmava_rollout.so: argument checks, handle life cycle and kernel enqueueing.
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"
#include "layout.h"

using namespace mava;

namespace {

int obs_dim(const mava_config_t &c) { return kObsFixed + c.n_agents; }

bool config_ok(const mava_config_t &c) {
  return c.grid >= 3 && c.grid <= 64 && c.n_agents >= 1 && c.n_agents <= kMaxAgents && c.n_food >= 1 &&
         c.n_food <= kMaxFood && c.max_agent_level >= 1 && c.max_agent_level <= 3 &&
         c.n_agents + c.n_food <= c.grid * c.grid && c.episode_cap >= 1 && c.n_envs >= 1 && c.max_T >= 1 &&
         c.hidden >= 1 && c.first_env >= 0 && c.env_kind >= 0 && c.env_kind <= 2 && (c.net_kind == MAVA_NET_SHARED_TORSO || c.net_kind == MAVA_NET_CENTRAL_CRITIC || c.net_kind == MAVA_NET_RECURRENT) &&
         (c.precision == MAVA_PRECISION_FP32 || c.precision == MAVA_PRECISION_BF16);
}

EnvParams env_params(const mava_rollout *h) {
  return EnvParams{h->cfg.grid, h->cfg.max_agent_level, h->cfg.episode_cap, h->cfg.n_envs, h->cfg.first_env,
                   static_cast<uint32_t>(h->cfg.seed), static_cast<uint32_t>(h->cfg.seed >> 32), h->cfg.env_kind};
}

struct DeviceGuard {  // makes the handle's device current for the duration of a call
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    ok = cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess);
    if (prev == dev) prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

// What an evaluation block adds to a launch (nullptr: a rollout).
struct EvalRequest {
  int32_t greedy;
  int32_t *count;
  float *ret;
  int32_t *len;
  int32_t *actions;
};

// `t_first`: the time row of the caller's buffers that step 0 of this launch writes (collect_host
// rolls a trajectory out in pieces).
int run_common(mava_rollout *h, const float *params_dev, int32_t T, const int32_t *forced, const EvalRequest *ev = nullptr,
               int32_t t_first = 0) {
  if (!h || !params_dev) return MAVA_ERR_INVALID_ARG;
  if (T < 1 || t_first < 0) return MAVA_ERR_INVALID_ARG;
  if (!ev && t_first + T > h->cfg.max_T) return MAVA_ERR_CAPACITY;  // an evaluation block stores no trajectory
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  RolloutArgs args{};
  args.env = env_params(h);
  args.buf = h->buf;
  if (t_first > 0) {  // rows t_first.. of every time-major array
    const size_t E = static_cast<size_t>(h->cfg.n_envs), M = E * h->cfg.n_agents, r0 = M * t_first;
    args.buf.obs += r0 * h->D; args.buf.actions += r0; args.buf.logp += r0; args.buf.values += r0;
    args.buf.rewards += r0; args.buf.dones += E * t_first;
    if (args.buf.logits) args.buf.logits += r0 * kActions;
  }
  args.state = h->d_state;
  args.forced = forced;
  args.T = T;
  args.t_global0 = h->t_global;
  args.write_logits = (h->cfg.flags & MAVA_FLAG_WRITE_LOGITS) ? 1 : 0;
  args.status = h->d_status;
  args.obs_last = h->d_obs_last;
  if (!ev && (h->expire_next & MAVA_EXPIRE_ROLLOUT) && h->cfg.precision == MAVA_PRECISION_BF16 && h->cfg.net_kind != MAVA_NET_RECURRENT &&
      tc_rollout_is_wide(h)) {
    args.debug_expire = 1;
    h->expire_next &= ~MAVA_EXPIRE_ROLLOUT;
  }
  if (ev) {
    args.eval = 1;
    args.greedy = ev->greedy;
    args.ev_count = ev->count; args.ev_ret = ev->ret; args.ev_len = ev->len; args.ev_actions = ev->actions;
    args.obs_last = nullptr;
  }
  cudaError_t err;
  if (h->cfg.net_kind == MAVA_NET_RECURRENT) {
    if (ev) return MAVA_ERR_UNSUPPORTED;  // no evaluation block for the recurrent policy
    err = h->cfg.precision == MAVA_PRECISION_BF16 ? launch_rollout_rec_tc(h, params_dev, args) : launch_rollout_rec_simt(h, params_dev, args);
  } else if (h->cfg.precision == MAVA_PRECISION_BF16) {
    err = launch_prep_tc(h, params_dev);
    if (err == cudaSuccess) err = launch_rollout_tc(h, args);
    if (err == cudaSuccess && !ev && h->cfg.net_kind == MAVA_NET_CENTRAL_CRITIC) err = launch_critic_tc(h, params_dev, T);
  } else {
    err = launch_prep_simt(h, params_dev);
    if (err == cudaSuccess) err = launch_rollout_simt(h, args);
  }
  if (err != cudaSuccess) return MAVA_ERR_CUDA;
  h->t_global += static_cast<uint32_t>(T);
  if (!ev) h->last_T = t_first + T;
  return MAVA_OK;
}

}  // namespace

extern "C" {

size_t mava_params_count(const mava_config_t *cfg) {
  if (!cfg || !config_ok(*cfg)) return 0;
  return param_layout(*cfg, obs_dim(*cfg), 1).total;
}

int32_t mava_state_record_len(const mava_config_t *cfg) {
  if (!cfg || !config_ok(*cfg)) return 0;
  return 3 * (cfg->n_agents + cfg->n_food) + 3;
}

int mava_rollout_create(const mava_config_t *cfg, const mava_buffers_t *buffers, void *cuda_stream,
                        mava_rollout_t **out) {
  if (!cfg || !buffers || !out) return MAVA_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(*cfg)) return MAVA_ERR_INVALID_ARG;
  if (cfg->view_radius != kViewRadius) return MAVA_ERR_UNSUPPORTED;
  if (cfg->n_agents * cfg->max_agent_level > 31) return MAVA_ERR_UNSUPPORTED;
  const mava_buffers_t &b = *buffers;
  if (!b.obs || !b.actions || !b.logp || !b.values || !b.rewards || !b.dones) return MAVA_ERR_INVALID_ARG;
  if ((cfg->flags & MAVA_FLAG_WRITE_LOGITS) && !b.logits) return MAVA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(b.obs) % 16 != 0) return MAVA_ERR_INVALID_ARG;
  const int variant = find_variant(*cfg);
  if (variant < 0) return MAVA_ERR_UNSUPPORTED;
  if (cfg->precision == MAVA_PRECISION_BF16 && !tc_supported(*cfg)) return MAVA_ERR_UNSUPPORTED;

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return MAVA_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MAVA_ERR_CUDA;
  if (prop.major != 10) return MAVA_ERR_UNSUPPORTED;  // kernels are built for sm_100a only

  mava_rollout *h = new (std::nothrow) mava_rollout();
  if (!h) return MAVA_ERR_CUDA;
  h->cfg = *cfg;
  h->buf = b;
  h->stream = static_cast<cudaStream_t>(cuda_stream);
  h->device = device;
  h->D = obs_dim(*cfg);
  h->variant = variant;
  const size_t np = param_layout(*cfg, h->D, 1).total;
  bool ok = cudaMalloc(&h->d_state, sizeof(EnvRec) * static_cast<size_t>(cfg->n_envs)) == cudaSuccess &&
            cudaMalloc(&h->d_status, sizeof(int)) == cudaSuccess &&
            cudaMalloc(&h->d_wsimt, sizeof(float) * simt_weight_floats(*cfg, h->D)) == cudaSuccess &&
            cudaMalloc(&h->d_params_stage, sizeof(float) * np) == cudaSuccess;
  if (ok && cfg->precision == MAVA_PRECISION_BF16)
    ok = cudaMalloc(&h->d_wtc, tc_weight_bytes(*cfg, h->D)) == cudaSuccess;
  if (ok && cfg->net_kind == MAVA_NET_RECURRENT) {
    const size_t bytes = sizeof(float) * static_cast<size_t>(cfg->n_envs) * cfg->n_agents * cfg->hidden;
    ok = cudaMalloc(&h->d_hidden, bytes) == cudaSuccess && cudaMemsetAsync(h->d_hidden, 0, bytes, h->stream) == cudaSuccess;
  }
  if (ok && cfg->precision == MAVA_PRECISION_BF16 && cfg->net_kind == MAVA_NET_CENTRAL_CRITIC)
    ok = cudaMalloc(&h->d_critic, critic_weight_bytes(*cfg)) == cudaSuccess &&
         cudaMalloc(&h->d_obs_last, sizeof(float) * static_cast<size_t>(cfg->n_envs) * cfg->n_agents * h->D) == cudaSuccess;
  if (ok) ok = cudaMemsetAsync(h->d_status, 0, sizeof(int), h->stream) == cudaSuccess;
  if (ok) ok = launch_env_init(h) == cudaSuccess;
  if (ok) ok = cudaStreamSynchronize(h->stream) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    mava_rollout_destroy(h);
    return MAVA_ERR_CUDA;
  }
  *out = h;
  return MAVA_OK;
}

int mava_rollout_run(mava_rollout_t *h, const float *params_dev, int32_t T) {
  return run_common(h, params_dev, T, nullptr);
}

int mava_rollout_run_forced(mava_rollout_t *h, const float *params_dev, int32_t T, const int32_t *actions_dev) {
  if (!actions_dev) return MAVA_ERR_INVALID_ARG;
  return run_common(h, params_dev, T, actions_dev);
}

int mava_rollout_evaluate(mava_rollout_t *h, const float *params_dev, int32_t T, int32_t greedy, int32_t *ep_count_dev,
                          float *ret_sum_dev, int32_t *len_sum_dev, int32_t *actions_dev) {
  if (!ep_count_dev || !ret_sum_dev || !len_sum_dev) return MAVA_ERR_INVALID_ARG;
  const EvalRequest ev{greedy ? 1 : 0, ep_count_dev, ret_sum_dev, len_sum_dev, actions_dev};
  return run_common(h, params_dev, T, nullptr, &ev);
}

int mava_gae(mava_rollout_t *h, float gamma, float lambda) {
  if (!h || h->last_T < 1 || !h->buf.adv || !h->buf.ret) return MAVA_ERR_INVALID_ARG;
  if (!(gamma >= 0.0f && gamma <= 1.0f && lambda >= 0.0f && lambda <= 1.0f)) return MAVA_ERR_INVALID_ARG;
  if (h->last_T > MAVA_GAE_MAX_T) return MAVA_ERR_CAPACITY;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  return launch_gae(h, gamma, lambda) == cudaSuccess ? MAVA_OK : MAVA_ERR_CUDA;
}

int mava_debug_expire_next_wait(mava_rollout_t *h, int32_t which) {
  if (!h || (which != MAVA_EXPIRE_GAE && which != MAVA_EXPIRE_ROLLOUT)) return MAVA_ERR_INVALID_ARG;
  h->expire_next |= which;
  return MAVA_OK;
}

void mava_ppo_defaults(mava_ppo_hyper_t *hp) {
  if (!hp) return;
  hp->clip_eps = 0.2f; hp->ent_coef = 0.01f; hp->vf_coef = 0.5f;
  hp->lr = 2.5e-4f; hp->beta1 = 0.9f; hp->beta2 = 0.999f; hp->adam_eps = 1e-5f;
  hp->max_grad_norm = 0.5f;
}

int mava_ppo_grad(mava_rollout_t *h, const float *params_dev, const mava_ppo_hyper_t *hp, float *grad_dev, float *terms_dev) {
  if (!h || !params_dev || !hp || !grad_dev || h->last_T < 1 || !h->buf.adv || !h->buf.ret) return MAVA_ERR_INVALID_ARG;
  if (!(hp->clip_eps > 0.0f)) return MAVA_ERR_INVALID_ARG;
  if (h->cfg.net_kind == MAVA_NET_RECURRENT) return MAVA_ERR_UNSUPPORTED;  // no update block for the recurrent policy
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  return launch_ppo_grad(h, params_dev, *hp, grad_dev, terms_dev, nullptr, 0) == cudaSuccess ? MAVA_OK : MAVA_ERR_CUDA;
}

int mava_ppo_grad_envs(mava_rollout_t *h, const float *params_dev, const mava_ppo_hyper_t *hp, const int32_t *env_ids_dev,
                       int32_t n_ids, float *grad_dev, float *terms_dev) {
  if (!h || !params_dev || !hp || !grad_dev || !env_ids_dev || n_ids < 1 || h->last_T < 1 || !h->buf.adv || !h->buf.ret)
    return MAVA_ERR_INVALID_ARG;
  if (!(hp->clip_eps > 0.0f)) return MAVA_ERR_INVALID_ARG;
  if (h->cfg.net_kind == MAVA_NET_RECURRENT) return MAVA_ERR_UNSUPPORTED;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  return launch_ppo_grad(h, params_dev, *hp, grad_dev, terms_dev, env_ids_dev, n_ids) == cudaSuccess ? MAVA_OK : MAVA_ERR_CUDA;
}

int mava_adam_step(mava_rollout_t *h, float *params_dev, const float *grad_dev, float *m_dev, float *v_dev, int32_t step,
                   const mava_ppo_hyper_t *hp) {
  if (!h || !params_dev || !grad_dev || !m_dev || !v_dev || !hp || step < 1) return MAVA_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  return launch_adam_step(h, params_dev, grad_dev, m_dev, v_dev, step, *hp) == cudaSuccess ? MAVA_OK : MAVA_ERR_CUDA;
}

int mava_ppo_update(mava_rollout_t *h, float *params_dev, float *m_dev, float *v_dev, float *grad_dev, const mava_ppo_hyper_t *hp,
                    int32_t epochs, int32_t minibatches, const int32_t *perm_dev, int32_t first_step, float *terms_dev) {
  if (!h || !params_dev || !m_dev || !v_dev || !grad_dev || !hp || !perm_dev || epochs < 1 || minibatches < 1 || first_step < 1 ||
      minibatches > h->cfg.n_envs)
    return MAVA_ERR_INVALID_ARG;
  const int E = h->cfg.n_envs;
  int step = first_step;
  for (int e = 0; e < epochs; ++e)
    for (int k = 0; k < minibatches; ++k) {
      const int lo = static_cast<int>(static_cast<int64_t>(E) * k / minibatches), hi = static_cast<int>(static_cast<int64_t>(E) * (k + 1) / minibatches);
      float *terms = terms_dev ? terms_dev + 4 * (static_cast<size_t>(e) * minibatches + k) : nullptr;
      int rc = mava_ppo_grad_envs(h, params_dev, hp, perm_dev + static_cast<size_t>(e) * E + lo, hi - lo, grad_dev, terms);
      if (rc == MAVA_OK) rc = mava_adam_step(h, params_dev, grad_dev, m_dev, v_dev, step++, hp);
      if (rc != MAVA_OK) return rc;
    }
  return MAVA_OK;
}

int mava_rollout_reset(mava_rollout_t *h, uint64_t seed) {
  if (!h) return MAVA_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  h->cfg.seed = seed;
  h->t_global = 0;
  h->last_T = 0;
  if (h->d_hidden &&
      cudaMemsetAsync(h->d_hidden, 0, sizeof(float) * static_cast<size_t>(h->cfg.n_envs) * h->cfg.n_agents * h->cfg.hidden, h->stream) != cudaSuccess)
    return MAVA_ERR_CUDA;
  return launch_env_init(h) == cudaSuccess ? MAVA_OK : MAVA_ERR_CUDA;
}

int mava_rollout_status(mava_rollout_t *h) {
  if (!h) return MAVA_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  int status = 0;
  if (cudaMemcpyAsync(&status, h->d_status, sizeof(int), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return MAVA_ERR_CUDA;
  if (status != 0) {
    cudaMemsetAsync(h->d_status, 0, sizeof(int), h->stream);
    return status == kStatusBadIndex ? MAVA_ERR_INVALID_ARG : MAVA_ERR_DEVICE_TIMEOUT;
  }
  return MAVA_OK;
}

int mava_rollout_get_state(mava_rollout_t *h, int32_t *records_host) {
  if (!h || !records_host) return MAVA_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  const int E = h->cfg.n_envs, N = h->cfg.n_agents, F = h->cfg.n_food;
  std::vector<EnvRec> recs(static_cast<size_t>(E));
  if (cudaMemcpyAsync(recs.data(), h->d_state, sizeof(EnvRec) * recs.size(), cudaMemcpyDeviceToHost, h->stream) !=
          cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return MAVA_ERR_CUDA;
  const int len = 3 * (N + F) + 3;
  for (int e = 0; e < E; ++e) {
    int32_t *o = records_host + static_cast<size_t>(e) * len;
    const EnvRec &s = recs[static_cast<size_t>(e)];
    for (int n = 0; n < N; ++n) { *o++ = s.ar[n]; *o++ = s.ac[n]; *o++ = s.al[n]; }
    for (int f = 0; f < F; ++f) { *o++ = s.fr[f]; *o++ = s.fc[f]; *o++ = s.fl[f]; }
    *o++ = s.step; *o++ = s.episode; *o++ = s.total;
  }
  return MAVA_OK;
}

int mava_rollout_set_state(mava_rollout_t *h, const int32_t *records_host) {
  if (!h || !records_host) return MAVA_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  const int E = h->cfg.n_envs, N = h->cfg.n_agents, F = h->cfg.n_food, G = h->cfg.grid;
  const int len = 3 * (N + F) + 3;
  std::vector<EnvRec> recs(static_cast<size_t>(E));
  for (int e = 0; e < E; ++e) {
    const int32_t *in = records_host + static_cast<size_t>(e) * len;
    EnvRec s{};
    for (int n = 0; n < N; ++n) {
      const int r = *in++, c = *in++, l = *in++;
      if (r < 0 || r >= G || c < 0 || c >= G) return MAVA_ERR_INVALID_ARG;
      if (h->cfg.env_kind == 0 ? (l < 1 || l > 3) : (l < 0 || l > F)) return MAVA_ERR_INVALID_ARG;
      s.ar[n] = static_cast<uint8_t>(r); s.ac[n] = static_cast<uint8_t>(c); s.al[n] = static_cast<uint8_t>(l);
    }
    for (int f = 0; f < F; ++f) {
      const int r = *in++, c = *in++, l = *in++;
      if (r < 0 || r >= G || c < 0 || c >= G || l < 0 || l > 31) return MAVA_ERR_INVALID_ARG;
      s.fr[f] = static_cast<uint8_t>(r); s.fc[f] = static_cast<uint8_t>(c); s.fl[f] = static_cast<uint8_t>(l);
    }
    s.step = *in++; s.episode = *in++; s.total = *in++;
    if (s.step < 0 || s.step >= h->cfg.episode_cap || s.episode < 0 || s.total < (h->cfg.env_kind == 0 ? 1 : 0)) return MAVA_ERR_INVALID_ARG;
    recs[static_cast<size_t>(e)] = s;
  }
  if (cudaStreamSynchronize(h->stream) != cudaSuccess ||
      cudaMemcpy(h->d_state, recs.data(), sizeof(EnvRec) * recs.size(), cudaMemcpyHostToDevice) != cudaSuccess)
    return MAVA_ERR_CUDA;
  return MAVA_OK;
}

int mava_rollout_get_hidden(mava_rollout_t *h, float *hidden_host) {
  if (!h || !hidden_host || !h->d_hidden) return MAVA_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  const size_t bytes = sizeof(float) * static_cast<size_t>(h->cfg.n_envs) * h->cfg.n_agents * h->cfg.hidden;
  if (cudaMemcpyAsync(hidden_host, h->d_hidden, bytes, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return MAVA_ERR_CUDA;
  return MAVA_OK;
}

int mava_rollout_collect_host(mava_rollout_t *h, const float *params_host, int32_t T, float gamma, float lambda,
                              const mava_host_buffers_t *out) {
  if (!h || !params_host || !out) return MAVA_ERR_INVALID_ARG;
  if (T < 1) return MAVA_ERR_INVALID_ARG;
  if (T > h->cfg.max_T || (h->buf.adv && h->buf.ret && T > MAVA_GAE_MAX_T)) return MAVA_ERR_CAPACITY;  // before anything is enqueued
  DeviceGuard guard(h->device);
  if (!guard.ok) return MAVA_ERR_CUDA;
  const size_t np = param_layout(h->cfg, h->D, 1).total;
  if (cudaMemcpyAsync(h->d_params_stage, params_host, np * sizeof(float), cudaMemcpyHostToDevice, h->stream) !=
      cudaSuccess)
    return MAVA_ERR_CUDA;
  if (!h->copy_ready) {
    bool made = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; made && i <= kCollectChunks; ++i)
      made = cudaEventCreateWithFlags(&h->chunk_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!made) return MAVA_ERR_CUDA;
    h->copy_ready = true;
  }
  // The copies are bound by the host link and take several times as long as the kernels, so the
  // rollout is cut into pieces in time (two calls continue like one) and the rows of a finished
  // piece travel while the next piece runs.  The centralised critic works on the whole trajectory
  // at once and is not cut.
  const int chunks = (h->cfg.net_kind == MAVA_NET_CENTRAL_CRITIC || T < 2 * kCollectChunks) ? 1 : kCollectChunks;
  const size_t E = static_cast<size_t>(h->cfg.n_envs), M = E * h->cfg.n_agents;
  bool ok = true;
  auto back = [&](void *dst, const void *src, size_t offset, size_t bytes) {
    if (dst && src && ok)
      ok = cudaMemcpyAsync(static_cast<unsigned char *>(dst) + offset, static_cast<const unsigned char *>(src) + offset, bytes,
                           cudaMemcpyDeviceToHost, h->copy_stream) == cudaSuccess;
  };
  for (int c = 0; c < chunks; ++c) {
    const int32_t t0 = static_cast<int32_t>(static_cast<int64_t>(T) * c / chunks);
    const int32_t t1 = static_cast<int32_t>(static_cast<int64_t>(T) * (c + 1) / chunks);
    const int rc = run_common(h, h->d_params_stage, t1 - t0, nullptr, nullptr, t0);
    if (rc != MAVA_OK) return rc;
    if (cudaEventRecord(h->chunk_done[c], h->stream) != cudaSuccess ||
        cudaStreamWaitEvent(h->copy_stream, h->chunk_done[c], 0) != cudaSuccess)
      return MAVA_ERR_CUDA;
    const size_t r0 = M * t0, rn = M * (t1 - t0);
    back(out->obs, h->buf.obs, r0 * h->D * sizeof(float), rn * h->D * sizeof(float));
    back(out->actions, h->buf.actions, r0 * sizeof(int32_t), rn * sizeof(int32_t));
    back(out->logp, h->buf.logp, r0 * sizeof(float), rn * sizeof(float));
    back(out->values, h->buf.values, r0 * sizeof(float), (rn + (c == chunks - 1 ? M : 0)) * sizeof(float));
    back(out->rewards, h->buf.rewards, r0 * sizeof(float), rn * sizeof(float));
    back(out->dones, h->buf.dones, E * t0, E * (t1 - t0));
    if (h->cfg.flags & MAVA_FLAG_WRITE_LOGITS)
      back(out->logits, h->buf.logits, r0 * kActions * sizeof(float), rn * kActions * sizeof(float));
  }
  if (h->buf.adv && h->buf.ret) {
    const int rc = mava_gae(h, gamma, lambda);
    if (rc != MAVA_OK) return rc;
    if (cudaEventRecord(h->chunk_done[kCollectChunks], h->stream) != cudaSuccess ||
        cudaStreamWaitEvent(h->copy_stream, h->chunk_done[kCollectChunks], 0) != cudaSuccess)
      return MAVA_ERR_CUDA;
    back(out->adv, h->buf.adv, 0, M * T * sizeof(float));
    back(out->ret, h->buf.ret, 0, M * T * sizeof(float));
  }
  if (!ok || cudaStreamSynchronize(h->copy_stream) != cudaSuccess || cudaStreamSynchronize(h->stream) != cudaSuccess)
    return MAVA_ERR_CUDA;
  return MAVA_OK;
}

int64_t mava_rollout_launch_count(const mava_rollout_t *h) { return h ? h->launches : 0; }

// ---- allocation-free variant ----------------------------------------------------------------
// Scratch of mava_rollout_run_static: every GPU that loads this library carries these bytes
// until the process exits.  In host code `g_static_scratch` is only a stand-in for the symbol;
// the device address comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[MAVA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
unsigned char *g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on `device` (which must be current), resolved on first use.
unsigned char *static_scratch(int device) {
  if (device < 0 || device >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[device]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    g_scratch_addr[device] = static_cast<unsigned char *>(ptr);
  }
  return g_scratch_addr[device];
}

size_t round256(size_t n) { return (n + 255) / 256 * 256; }
}  // namespace

int mava_rollout_run_static(const mava_config_t *cfg, const mava_buffers_t *buffers, const float *params_dev,
                            int32_t T, void *cuda_stream) {
  if (!cfg || !buffers || !params_dev) return MAVA_ERR_INVALID_ARG;
  if (!config_ok(*cfg) || T < 1) return MAVA_ERR_INVALID_ARG;
  if (T > cfg->max_T) return MAVA_ERR_CAPACITY;
  if (cfg->view_radius != kViewRadius || cfg->n_agents * cfg->max_agent_level > 31) return MAVA_ERR_UNSUPPORTED;
  const mava_buffers_t &b = *buffers;
  if (!b.obs || !b.actions || !b.logp || !b.values || !b.rewards || !b.dones) return MAVA_ERR_INVALID_ARG;
  if ((cfg->flags & MAVA_FLAG_WRITE_LOGITS) && !b.logits) return MAVA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(b.obs) % 16 != 0) return MAVA_ERR_INVALID_ARG;
  const int variant = find_variant(*cfg);
  if (variant < 0) return MAVA_ERR_UNSUPPORTED;
  const bool bf16 = cfg->precision == MAVA_PRECISION_BF16;
  if (cfg->net_kind == MAVA_NET_RECURRENT) return MAVA_ERR_UNSUPPORTED;  // its hidden vectors are handle state
  if (bf16 && !tc_supported(*cfg)) return MAVA_ERR_UNSUPPORTED;
  if (bf16 && cfg->net_kind == MAVA_NET_CENTRAL_CRITIC) return MAVA_ERR_UNSUPPORTED;  // its scratch is far beyond the array

  // carve the scratch: status word | environment states | re-laid-out weights
  const int D = obs_dim(*cfg);
  const size_t state_bytes = round256(sizeof(EnvRec) * static_cast<size_t>(cfg->n_envs));
  const size_t weight_bytes = round256(bf16 ? tc_weight_bytes(*cfg, D) : sizeof(float) * simt_weight_floats(*cfg, D));
  if (256 + state_bytes + weight_bytes > MAVA_STATIC_SCRATCH_BYTES) return MAVA_ERR_CAPACITY;

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return MAVA_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return MAVA_ERR_CUDA;
  if (major != 10) return MAVA_ERR_UNSUPPORTED;
  unsigned char *scratch = static_scratch(device);
  if (!scratch) return MAVA_ERR_CUDA;

  mava_rollout h{};  // a handle on the stack whose device state lives in the static array
  h.cfg = *cfg;
  h.buf = b;
  h.stream = static_cast<cudaStream_t>(cuda_stream);
  h.device = device;
  h.D = D;
  h.variant = variant;
  h.d_status = reinterpret_cast<int *>(scratch);
  h.d_state = reinterpret_cast<EnvRec *>(scratch + 256);
  if (bf16) h.d_wtc = scratch + 256 + state_bytes;
  else h.d_wsimt = reinterpret_cast<float *>(scratch + 256 + state_bytes);

  // the array keeps what the previous call left: the status word must start at zero; the
  // states and the weights are fully rewritten by the kernels below
  if (cudaMemsetAsync(h.d_status, 0, sizeof(int), h.stream) != cudaSuccess) return MAVA_ERR_CUDA;
  if (launch_env_init(&h) != cudaSuccess) return MAVA_ERR_CUDA;
  const int rc = run_common(&h, params_dev, T, nullptr);
  if (rc != MAVA_OK) return rc;
  int status = 0;
  if (cudaMemcpyAsync(&status, h.d_status, sizeof(int), cudaMemcpyDeviceToHost, h.stream) != cudaSuccess ||
      cudaStreamSynchronize(h.stream) != cudaSuccess)
    return MAVA_ERR_CUDA;
  return status != 0 ? MAVA_ERR_DEVICE_TIMEOUT : MAVA_OK;
}

void mava_rollout_destroy(mava_rollout_t *h) {
  if (!h) return;
  DeviceGuard guard(h->device);
  cudaStreamSynchronize(h->stream);
  cudaFree(h->d_state);
  cudaFree(h->d_status);
  cudaFree(h->d_wsimt);
  cudaFree(h->d_wtc);
  cudaFree(h->d_params_stage);
  cudaFree(h->d_critic);
  cudaFree(h->d_obs_last);
  cudaFree(h->d_upd);
  cudaFree(h->d_upd_stage);
  cudaFree(h->d_hidden);
  if (h->copy_ready) {
    cudaStreamSynchronize(h->copy_stream);
    for (int i = 0; i <= kCollectChunks; ++i) cudaEventDestroy(h->chunk_done[i]);
    cudaStreamDestroy(h->copy_stream);
  }
  delete h;
}

const char *mava_strerror(int code) {
  switch (code) {
    case MAVA_OK: return "ok";
    case MAVA_ERR_INVALID_ARG: return "invalid argument";
    case MAVA_ERR_UNSUPPORTED: return "unsupported configuration or device";
    case MAVA_ERR_CUDA: return "CUDA runtime error";
    case MAVA_ERR_DEVICE_TIMEOUT: return "a device-side bounded wait gave up";
    case MAVA_ERR_CAPACITY: return "size beyond the stated capacity";
    default: return "unknown error";
  }
}

}  // extern "C"
