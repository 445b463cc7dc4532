// fp32 SIMT rollout: one CTA owns a tile of environments for all T steps; the environment
// states, the observation tile and the hidden activations stay in shared memory, the weights
// (transposed to [in][out]) are read through L1/L2.  This is the validation path: plain FMA
// arithmetic in index order, no tensor cores.
#include "common.cuh"
#include "env.cuh"
#include "env_wh.cuh"
#include "layout.h"
#include "simt_dense.cuh"

namespace mava {

namespace {

template <int N, int F, int H, bool CENTRAL>
struct SimtSmem {
  static constexpr int D = kObsFixed + N;
  static constexpr int EPT = kSimtRows / N;  // environments per tile
  static constexpr int HS = H + 1;           // padded stride of the hidden buffers
  EnvRec st[EPT];
  alignas(16) float obs[kSimtRows * D];      // [row][D], rows of one env are contiguous
  float h1[kSimtRows * HS];
  float h2[kSimtRows * HS];
  float logits[kSimtRows * 8];
  float value[kSimtRows];
  int act[kSimtRows];
  uint8_t new_r[kSimtRows], new_c[kSimtRows], collected[EPT * F];
};

// ENV: 0 foraging, 1 warehouse (env_wh.cuh).
template <int N, int F, int H, bool CENTRAL, int ENV = 0>
__global__ void __launch_bounds__(kSimtThreads)
rollout_simt_kernel(RolloutArgs a, SimtWeights w) {
  using S = SimtSmem<N, F, H, CENTRAL>;
  constexpr int D = S::D, EPT = S::EPT, HS = S::HS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  S &sm = *reinterpret_cast<S *>(smem_raw);
  const int tid = threadIdx.x;
  const int e0 = blockIdx.x * EPT;
  const int n_env = min(EPT, a.env.n_envs - e0);
  if (n_env <= 0) return;
  const int n_rows = n_env * N;
  const size_t M = static_cast<size_t>(a.env.n_envs) * N;

  for (int i = tid; i < n_env * static_cast<int>(sizeof(EnvRec) / 4); i += kSimtThreads)
    reinterpret_cast<uint32_t *>(sm.st)[i] = reinterpret_cast<const uint32_t *>(a.state + e0)[i];
  for (int i = tid; i < kSimtRows * D; i += kSimtThreads) sm.obs[i] = 0.0f;
  __syncthreads();

  const bool ev = a.eval != 0;
  EvalSums sums;  // thread tid < n_env: environment e0 + tid
  for (int t = 0; t <= (ev ? a.T - 1 : a.T); ++t) {
    const bool last = !ev && (t == a.T);
    const size_t row0 = static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N;
    if constexpr (ENV == 0) {
      auto sink = [&](int row, int j, float v) { sm.obs[row * D + j] = v; };
      observe_fill<N>(sm.st, a.env, n_rows, tid, kSimtThreads, sink);
      __syncthreads();
      observe_scatter<N, F>(sm.st, n_rows, tid, kSimtThreads, sink);
    } else {
      for (int i = tid; i < n_rows * D; i += kSimtThreads) {
        const int row = i / D;
        sm.obs[i] = wh_obs_element<N, F>(sm.st[row / N], a.env, row % N, i - row * D);
      }
    }
    __syncthreads();

    if (!last && !ev) {  // the tile's rows are one contiguous block of the time-major obs array
      float *dst = a.buf.obs + row0 * D;
      const int count = n_rows * D;
      if (((row0 * D) & 3) == 0 && (count & 3) == 0) {
        for (int i = tid; i < count / 4; i += kSimtThreads)
          reinterpret_cast<float4 *>(dst)[i] = reinterpret_cast<const float4 *>(sm.obs)[i];
      } else {
        for (int i = tid; i < count; i += kSimtThreads) dst[i] = sm.obs[i];
      }
    }
    dense_tile<D, H, kSimtRows, true>(sm.obs, D, w.W1t, w.b1, sm.h1, HS, tid);
    __syncthreads();
    dense_tile<H, H, kSimtRows, true>(sm.h1, HS, w.W2t, w.b2, sm.h2, HS, tid);
    __syncthreads();
    {  // heads: one thread per (row, output)
      constexpr int OUTS = CENTRAL ? kActions : kActions + 1;
      if (tid < kSimtRows * OUTS) {
        const int row = tid / OUTS, o = tid - row * OUTS;
        const float *wrow = (o < kActions) ? w.Wa + o * H : w.Wv;
        float acc = 0.0f;
        for (int k = 0; k < H; ++k) acc = fmaf(sm.h2[row * HS + k], __ldg(wrow + k), acc);
        if (o < kActions) sm.logits[row * 8 + o] = acc + __ldg(w.ba + o);
        else sm.value[row] = acc + __ldg(w.bv);
      }
    }
    __syncthreads();
    if constexpr (CENTRAL) {  // critic on the concatenated observations of each environment
      dense_tile<N * D, H, EPT, true>(sm.obs, N * D, w.C1t, w.c1, sm.h1, HS, tid);
      __syncthreads();
      dense_tile<H, H, EPT, true>(sm.h1, HS, w.C2t, w.c2, sm.h2, HS, tid);
      __syncthreads();
      if (tid < EPT) {
        float acc = 0.0f;
        for (int k = 0; k < H; ++k) acc = fmaf(sm.h2[tid * HS + k], __ldg(w.Cv + k), acc);
        acc += __ldg(w.cv);
        for (int n = 0; n < N; ++n) sm.value[tid * N + n] = acc;
      }
      __syncthreads();
    }

    if (tid < n_rows) {
      if (!ev) a.buf.values[row0 + tid] = sm.value[tid];
      if (!last) {
        const int le = tid / N, ag = tid - le * N;
        float l[kActions], e[kActions];
        float m = sm.logits[tid * 8];
#pragma unroll
        for (int k = 0; k < kActions; ++k) { l[k] = sm.logits[tid * 8 + k]; m = fmaxf(m, l[k]); }
        float sum = 0.0f;
#pragma unroll
        for (int k = 0; k < kActions; ++k) { e[k] = expf(l[k] - m); sum += e[k]; }
        const float u = action_uniform(a.env, a.t_global0 + static_cast<uint32_t>(t),
                                       static_cast<uint32_t>(a.env.first_env + e0 + le), static_cast<uint32_t>(ag));
        const float target = u * sum;
        int action = kActions - 1;
        float cdf = 0.0f;
        bool found = false;
#pragma unroll
        for (int k = 0; k < kActions; ++k) {
          cdf += e[k];
          if (!found && target < cdf) { action = k; found = true; }
        }
        if (a.forced) {
          action = a.forced[row0 + tid];
          if (action < 0 || action >= kActions) action = 0;
        }
        if (ev && a.greedy) action = greedy_action(l);
        float la = l[0];
#pragma unroll
        for (int k = 1; k < kActions; ++k) la = (action == k) ? l[k] : la;
        sm.act[tid] = action;
        if (ev) {
          if (a.ev_actions) a.ev_actions[row0 + tid] = action;
        } else {
          a.buf.actions[row0 + tid] = action;
          a.buf.logp[row0 + tid] = la - m - logf(sum);
          if (a.write_logits) {
#pragma unroll
            for (int k = 0; k < kActions; ++k) a.buf.logits[(row0 + tid) * kActions + k] = l[k];
          }
        }
      }
    }
    __syncthreads();
    if (last) break;

    if constexpr (ENV == 0) {
      step_decide<N, F>(sm.st, a.env, sm.act, n_env, sm.new_r, sm.new_c, sm.collected, tid, kSimtThreads);
      __syncthreads();
    }
    if (tid < n_env) {
      float reward;
      bool done;
      if constexpr (ENV == 0)
        step_apply<N, F>(sm.st[tid], a.env, static_cast<uint32_t>(a.env.first_env + e0 + tid), sm.new_r, sm.new_c,
                         sm.collected, tid, reward, done);
      else
        wh_step_rec<N, F>(sm.st[tid], a.env, static_cast<uint32_t>(a.env.first_env + e0 + tid), sm.act + tid * N, reward, done);
      if (ev) {
        sums.step(reward, done);
      } else {
        for (int n = 0; n < N; ++n) a.buf.rewards[row0 + tid * N + n] = reward;
        a.buf.dones[static_cast<size_t>(t) * a.env.n_envs + e0 + tid] = done ? 1 : 0;
      }
    }
    __syncthreads();
  }
  if (ev && tid < n_env) {
    a.ev_count[e0 + tid] = sums.count; a.ev_ret[e0 + tid] = sums.ret; a.ev_len[e0 + tid] = sums.len;
  }

  for (int i = tid; i < n_env * static_cast<int>(sizeof(EnvRec) / 4); i += kSimtThreads)
    reinterpret_cast<uint32_t *>(a.state + e0)[i] = reinterpret_cast<const uint32_t *>(sm.st)[i];
}

template <int N, int F>
__global__ void env_init_kernel(EnvRec *state, EnvParams p) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= p.n_envs) return;
  EnvRec s;
  memset(&s, 0, sizeof(s));
  if (p.env_kind == 0) env_reset<N, F>(s, p, static_cast<uint32_t>(p.first_env + e), 0u);
  else wh_reset_rec<N, F>(s, p, static_cast<uint32_t>(p.first_env + e), 0u);
  state[e] = s;
}

// Transposes the [out][in] weight matrices of the hidden layers to [in][out] and copies the rest.
__global__ void prep_simt_kernel(const float *__restrict__ src, float *__restrict__ dst, ParamLayout in,
                                 ParamLayout out, int D, int H, int N, int central) {
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  auto transpose = [&](size_t s, size_t d, int rows_out, int cols_in) {
    const size_t n = static_cast<size_t>(rows_out) * cols_in;
    for (size_t i = tid; i < n; i += stride) {
      const size_t k = i / rows_out, o = i - k * rows_out;  // dst index i = k*rows_out + o
      dst[d + i] = src[s + o * cols_in + k];
    }
  };
  auto copy = [&](size_t s, size_t d, size_t n) {
    for (size_t i = tid; i < n; i += stride) dst[d + i] = src[s + i];
  };
  transpose(in.W1, out.W1, H, D); copy(in.b1, out.b1, H);
  transpose(in.W2, out.W2, H, H); copy(in.b2, out.b2, H);
  copy(in.Wa, out.Wa, static_cast<size_t>(kActions) * H); copy(in.ba, out.ba, kActions);
  if (!central) {
    copy(in.Wv, out.Wv, H); copy(in.bv, out.bv, 1);
  } else {
    transpose(in.C1, out.C1, H, N * D); copy(in.c1, out.c1, H);
    transpose(in.C2, out.C2, H, H); copy(in.c2, out.c2, H);
    copy(in.Cv, out.Cv, H); copy(in.cv, out.cv, 1);
  }
}

template <int N, int F, int H, bool CENTRAL, int ENV = 0>
cudaError_t launch_simt_variant(mava_rollout *h, const RolloutArgs &args, const SimtWeights &w) {
  using S = SimtSmem<N, F, H, CENTRAL>;
  auto kern = rollout_simt_kernel<N, F, H, CENTRAL, ENV>;
  const size_t smem = sizeof(S);
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  const int tiles = (h->cfg.n_envs + S::EPT - 1) / S::EPT;
  kern<<<tiles, kSimtThreads, smem, h->stream>>>(args, w);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace

// The compiled (N, F, H, net_kind) combinations.
int find_variant(const mava_config_t &c) {
  struct V { int n, f, h, kind; };
  static const V table[] = {{2, 2, 64, 0}, {2, 2, 128, 0}, {3, 3, 128, 0}, {4, 5, 256, 1}, {8, 8, 256, 0},
                            {2, 2, 64, 2}, {3, 3, 64, 2}};  // the last two: the recurrent policy
  for (int i = 0; i < 7; ++i)
    if (table[i].n == c.n_agents && table[i].f == c.n_food && table[i].h == c.hidden && table[i].kind == c.net_kind)
      return i;
  return -1;
}

size_t simt_weight_floats(const mava_config_t &cfg, int D) { return param_layout(cfg, D, 4).total; }

cudaError_t launch_env_init(mava_rollout *h) {
  EnvParams p{h->cfg.grid, h->cfg.max_agent_level, h->cfg.episode_cap, h->cfg.n_envs, h->cfg.first_env,
              static_cast<uint32_t>(h->cfg.seed), static_cast<uint32_t>(h->cfg.seed >> 32), h->cfg.env_kind};
  const int threads = 128, blocks = (h->cfg.n_envs + threads - 1) / threads;
  switch (h->variant) {
    case 0: case 1: case 5: env_init_kernel<2, 2><<<blocks, threads, 0, h->stream>>>(h->d_state, p); break;
    case 2: case 6: env_init_kernel<3, 3><<<blocks, threads, 0, h->stream>>>(h->d_state, p); break;
    case 3: env_init_kernel<4, 5><<<blocks, threads, 0, h->stream>>>(h->d_state, p); break;
    case 4: env_init_kernel<8, 8><<<blocks, threads, 0, h->stream>>>(h->d_state, p); break;
    default: return cudaErrorInvalidValue;
  }
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_prep_simt(mava_rollout *h, const float *params_dev) {
  const ParamLayout in = param_layout(h->cfg, h->D, 1), out = param_layout(h->cfg, h->D, 4);
  prep_simt_kernel<<<148, 256, 0, h->stream>>>(params_dev, h->d_wsimt, in, out, h->D, h->cfg.hidden,
                                               h->cfg.n_agents, h->cfg.net_kind == MAVA_NET_CENTRAL_CRITIC);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_rollout_simt(mava_rollout *h, const RolloutArgs &args) {
  const ParamLayout L = param_layout(h->cfg, h->D, 4);
  const float *base = h->d_wsimt;
  SimtWeights w{};
  w.W1t = base + L.W1; w.b1 = base + L.b1; w.W2t = base + L.W2; w.b2 = base + L.b2;
  w.Wa = base + L.Wa; w.ba = base + L.ba;
  if (h->cfg.net_kind == MAVA_NET_SHARED_TORSO) {
    w.Wv = base + L.Wv; w.bv = base + L.bv;
  } else {
    w.Wv = base + L.Cv; w.bv = base + L.cv;  // unused by the head loop of the central variant
    w.C1t = base + L.C1; w.c1 = base + L.c1; w.C2t = base + L.C2; w.c2 = base + L.c2;
    w.Cv = base + L.Cv; w.cv = base + L.cv;
  }
  if (h->cfg.env_kind != 0) {  // the warehouse family is compiled for two shapes
    switch (h->variant) {
      case 0: return launch_simt_variant<2, 2, 64, false, 1>(h, args, w);
      case 2: return launch_simt_variant<3, 3, 128, false, 1>(h, args, w);
      default: return cudaErrorNotSupported;
    }
  }
  switch (h->variant) {
    case 0: return launch_simt_variant<2, 2, 64, false>(h, args, w);
    case 1: return launch_simt_variant<2, 2, 128, false>(h, args, w);
    case 2: return launch_simt_variant<3, 3, 128, false>(h, args, w);
    case 3: return launch_simt_variant<4, 5, 256, true>(h, args, w);
    case 4: return launch_simt_variant<8, 8, 256, false>(h, args, w);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace mava
